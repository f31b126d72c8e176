// Tensor-core prefill kernels: bf16, d = 128, S = 64, G = 4, any local window of up to 16 chunks (W <= 897), one
// landmark per KV head or per query head (the latter with K <= 32: the tcgen05 selection kernel).
//
// With independent queries the tokens that select a chunk are scattered over the sequence, so the
// path is organised CHUNK-MAJOR: K/V of a chunk are staged once and reused by every query row that
// selected it; what moves per (token, chunk) pair is the query rows in and one bf16 output row out.
//
//   prefill_select  warp-MMA scoring + top-K, the fallback for K > 32 (the tcgen05 kernel lives in
//                   prefill_select_tc.cu): per (sequence, KV head, 64-token tile) it streams landmark tiles
//                   through a TMA ring, scores them for the 4 heads (Eq. surrogate top-k), takes the group
//                   max (App. C) and keeps an exact running top-K per token (ties: lower chunk id).
//   invert_*        turn sel_idx into per-(query block, pair, chunk) lists of (token, slot) entries, every list
//                   starting on a tile boundary, the table of attend tiles, and the (token, slot) -> entry map.
//   (prefill_attend_tc.cu: the tcgen05 attend kernel over that tile table; one normalised bf16 output row
//                   and the per-head chunk mass per entry, in entry order.)
//   prefill_fuse    per (token, KV head): the softmax over {surrogate scores} U {log Z_swa}
//                   (Eq. HiLS weights) that mixes the rows written by the attend kernel.
#include "internal.h"
#include "tma.cuh"

namespace hils {
namespace {

constexpr int kD = 128;
constexpr int kS = 64;
constexpr int kG = 4;
constexpr int kQBDefault = 4096;             // tokens per pass of the invert/attend/fuse phases: the block's
                                             // queries (QB x 32 heads x 256 B = 32 MB) stay L2-resident while
                                             // they are gathered once per selected chunk
constexpr int kSelStages = 3;
constexpr int kSelStageBytes = kS * kD * 2;  // 64 landmark rows
constexpr float kLog2e = 1.4426950408889634f;

struct PArgs {
    Shape s;
    const __nv_bfloat16* q;
    const __nv_bfloat16* lm;
    const float* bias;
    __nv_bfloat16* out;
    float* lse;
    int32_t* sel;
    int* status;
    // scratch (per token block)
    int* cnt;               // [n_blocks*pairs*nc] rows of each (block, pair, chunk): selectors + own tokens
    int* cursor;            // [pairs*C]
    int* blk_toff;          // [n_blocks + 1] first tile of every query block (tiles are grouped by block)
    int* seg_tiles;         // [ceil(lists / 1024)] tiles of each segment of 1024 lists
    int* off;               // [n_blocks*pairs*nc] first entry of each list; every list starts on a tile boundary
    int* entries;           // [max_tiles * tile_tok] (token_local << 8) | slot, grouped by (block, pair, chunk);
                            // slot K marks the token's own chunk (local branch); list tails up to the next tile
                            // boundary are padding
    int* epos;              // [pairs*L*(K+1)] entry index of every (token, slot), -1 = slot unused
    int4* tiles;            // [max_tiles] {pair, chunk, first entry, rows}
    __nv_bfloat16* obuf;    // [entries of one block][G][128] normalised per-chunk outputs, in entry order
    float* lam;             // [entries of one block][G] per-head surrogate scores; local slot: log Z_swa
    int i0, i1;             // token block [i0, i1) of the attend / fuse launch
    int blk;                // its index
    int n_blocks;           // query blocks of qb tokens
    int qb;                 // tokens per block the obuf / lam strides are sized for
    int nc;                 // chunk slots per pair in cnt/off/...: max(C, ceil(L / S))
    int tile_tok;           // entries per attend tile
    int max_tiles;
    int whole;              // obuf / lam cover all query blocks (indexed by global entry): one fuse launch per call
};

// ------------------------------------------------------------------------------------------ select
// Insert `key` into the unsorted K-entry list of one token (all 4 lanes of a quad call this with the
// same key).  tau / pmin track the smallest kept key (the K-th best so far) once the list is full.
__device__ __forceinline__ void quad_insert(unsigned long long* list, int K, int& cnt, unsigned long long& tau,
                                            int& pmin, unsigned long long key, int t, unsigned qmask) {
    if (cnt < K) {
        if (t == 0) list[cnt] = key;
        ++cnt;
        if (cnt < K) return;
    } else {
        if (t == 0) list[pmin] = key;
    }
    __syncwarp(qmask);
    unsigned long long mn = ~0ull;
    int pm = 0;
    for (int e = t; e < K; e += 4) {
        const unsigned long long x = list[e];
        if (x < mn) { mn = x; pm = e; }
    }
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
        const unsigned long long om = __shfl_xor_sync(qmask, mn, o);
        const int op = __shfl_xor_sync(qmask, pm, o);
        if (om < mn) { mn = om; pm = op; }
    }
    tau = mn;
    pmin = pm;
    __syncwarp(qmask);
}

struct SelSmem {
    uint64_t full[kSelStages];
    uint64_t empty[kSelStages];
};

__global__ void __launch_bounds__(160, 1)
prefill_select_kernel(const __grid_constant__ CUtensorMap map_lm, const PArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    SelSmem& sm = *reinterpret_cast<SelSmem*>(ring + kSelStages * kSelStageBytes);
    unsigned long long* lists = reinterpret_cast<unsigned long long*>(ring + kSelStages * kSelStageBytes + 64);

    const Shape& s = a.s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int pairs = s.B * s.Hkv;
    const int tiles_per_seq = (s.R + kS - 1) / kS;
    const int ci = tiles_per_seq - 1 - static_cast<int>(blockIdx.x) / pairs;      // heavy tiles first
    const int pair = static_cast<int>(blockIdx.x) % pairs;
    const int b = pair / s.Hkv, gk = pair % s.Hkv;
    // candidates of a token = the chunks left of its local window (Sec. 2.1); the tile's last token has the most
    const int ncand = local_lo(s.pos0 + min(s.R, (ci + 1) * kS) - 1, s.W, kS) / kS;
    const int nst = (ncand + kS - 1) / kS;
    const int K = s.K, Kp = K + 1;

    if (tid == 0) {
        for (int i = 0; i < kSelStages; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], 4); }
        mbar_fence_init();
        tma_prefetch_desc(&map_lm);
    }
    __syncthreads();

    if (warp == 4) {
        if (lane == 0) {
            for (int it = 0; it < nst; ++it) {
                const int st = it % kSelStages;
                if (it >= kSelStages && !mbar_wait(&sm.empty[st], ((it / kSelStages) - 1) & 1)) {
                    set_status(a.status, kDevTimeout);
                    break;
                }
                uint8_t* dst = ring + st * kSelStageBytes;
                const int row = pair * s.C + it * kS;
                mbar_expect_tx(&sm.full[st], kSelStageBytes);
                tma_load_2d(dst, &map_lm, &sm.full[st], 0, row);
                tma_load_2d(dst + 8192, &map_lm, &sm.full[st], 64, row);
            }
        }
        return;
    }

    const int g = lane >> 2, t = lane & 3;
    const unsigned qmask = 0xfu << (lane & ~3);
    const int tokA = ci * kS + warp * 16 + g, tokB = tokA + 8;
    const int ldA = min(tokA, s.R - 1), ldB = min(tokB, s.R - 1);
    const int ncA = local_lo(s.pos0 + ldA, s.W, kS) / kS, ncB = local_lo(s.pos0 + ldB, s.W, kS) / kS;

    // A operands: this warp's 16 tokens, one fragment set per head of the group
    uint32_t aq[kG][8][4];
#pragma unroll
    for (int h = 0; h < kG; ++h) {
        const __nv_bfloat16* qh = a.q + (static_cast<long long>(b) * s.Hq + gk * kG + h) * s.R * kD;
        const __nv_bfloat16* ra = qh + static_cast<long long>(ldA) * kD;
        const __nv_bfloat16* rb = qh + static_cast<long long>(ldB) * kD;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            aq[h][ks][0] = *reinterpret_cast<const uint32_t*>(ra + ks * 16 + 2 * t);
            aq[h][ks][1] = *reinterpret_cast<const uint32_t*>(rb + ks * 16 + 2 * t);
            aq[h][ks][2] = *reinterpret_cast<const uint32_t*>(ra + ks * 16 + 8 + 2 * t);
            aq[h][ks][3] = *reinterpret_cast<const uint32_t*>(rb + ks * 16 + 8 + 2 * t);
        }
    }
    unsigned long long* listA = lists + static_cast<size_t>(warp * 16 + g) * Kp;
    unsigned long long* listB = lists + static_cast<size_t>(warp * 16 + g + 8) * Kp;
    int cntA = 0, cntB = 0, pminA = 0, pminB = 0;
    unsigned long long tauA = 0ull, tauB = 0ull;
    const float* bias = a.bias ? a.bias + static_cast<long long>(pair) * s.C : nullptr;
    bool dead = false;

    for (int it = 0; it < nst && !dead; ++it) {
        const int st = it % kSelStages;
        if (!mbar_wait(&sm.full[st], (it / kSelStages) & 1)) {
            if (lane == 0) set_status(a.status, kDevTimeout);
            dead = true;
            break;
        }
        const uint32_t lm_addr = smem_u32(ring + st * kSelStageBytes);
        const int c0 = it * kS;
        const int ntl = min(8, (ncand - c0 + 7) >> 3);
        for (int nt = 0; nt < ntl; ++nt) {
            uint32_t bf[8][2];
#pragma unroll
            for (int kp = 0; kp < 4; ++kp) {
                const int row = nt * 8 + (lane & 7);
                const int dim = kp * 32 + (lane >> 3) * 8;
                ldmatrix_x4(lm_addr + (dim >> 6) * 8192 + swz128(row, (dim & 63) >> 3), bf[2 * kp][0], bf[2 * kp][1],
                            bf[2 * kp + 1][0], bf[2 * kp + 1][1]);
            }
            float um[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int h = 0; h < kG; ++h) {
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) mma_bf16_16816(acc, aq[h][ks], bf[ks][0], bf[ks][1]);
#pragma unroll
                for (int v = 0; v < 4; ++v) um[v] = fmaxf(um[v], acc[v]);
            }
            // um[0..1]: token A, chunks cb, cb+1; um[2..3]: token B
            const int cb = c0 + nt * 8 + 2 * t;
            unsigned long long key[4];
            bool any = false;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const int c = cb + (v & 1);
                const int nc_tok = v < 2 ? ncA : ncB;
                float u = um[v] * s.scale;
                if (bias && c < nc_tok) u += bias[c];
                key[v] = c < nc_tok ? select_key(u, c) : 0ull;
                any |= key[v] > ((v < 2) ? tauA : tauB);
            }
            if (__ballot_sync(kFullMask, any) == 0u) continue;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const bool pass = key[v] > ((v < 2) ? tauA : tauB);
                unsigned nib = (__ballot_sync(kFullMask, pass) >> (lane & ~3)) & 0xfu;
                while (nib) {
                    const int src = __ffs(nib) - 1;
                    nib &= nib - 1;
                    const unsigned long long x = __shfl_sync(qmask, key[v], (lane & ~3) + src);
                    if (v < 2) {
                        if (x > tauA) quad_insert(listA, K, cntA, tauA, pminA, x, t, qmask);
                    } else {
                        if (x > tauB) quad_insert(listB, K, cntB, tauB, pminB, x, t, qmask);
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.empty[st]);
    }

    // ascending chunk ids, -1 padded
    __syncwarp();
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        const int tok = half == 0 ? tokA : tokB;
        const unsigned long long* list = half == 0 ? listA : listB;
        const int n = half == 0 ? cntA : cntB;
        if (tok >= s.R) continue;
        int32_t* sel = a.sel + ((static_cast<long long>(pair)) * s.R + tok) * K;
        for (int e = t; e < n; e += 4) {
            const int id = key_chunk(list[e]);
            int rank = 0;
            for (int j = 0; j < n; ++j) rank += key_chunk(list[j]) < id ? 1 : 0;
            sel[rank] = id;
        }
        for (int e = n + t; e < K; e += 4) sel[e] = -1;
    }
}

// ------------------------------------------------------------------------------------------ invert
// Slots of a token: 0..K-1 the selected chunks, K..K+nl-1 the chunks of its local window [l(i), i] (Sec. 2.1:
// l(i) is chunk-aligned, so the window is whole chunks plus the causal part of the token's own chunk).  Every
// local chunk is attended like a selected one, with its own softmax; its chunk mass is the exact log-sum-exp of
// its scores, so the softmax over all slots' masses reproduces the single softmax over the window (Eq. chunk mass).
__host__ __device__ inline int max_local_slots(int W) { return (W - 1 + kS - 1) / kS + 1; }
__device__ __forceinline__ int slot_chunk(const PArgs& a, int pair, int tok, int slot) {
    if (slot >= a.s.K) {
        const int pos = a.s.pos0 + tok;
        const int c = local_lo(pos, a.s.W, kS) / kS + (slot - a.s.K);
        return c <= pos / kS ? c : -1;
    }
    return a.sel[(static_cast<long long>(pair) * a.s.R + tok) * a.s.K + slot];
}

__global__ void invert_count_kernel(const PArgs a) {
    const Shape& s = a.s;
    const int K1 = s.K + max_local_slots(s.W), pairs = s.B * s.Hkv;
    const long long total = static_cast<long long>(pairs) * s.R * K1;
    for (long long x = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; x < total;
         x += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int slot = static_cast<int>(x % K1);
        const int tok = static_cast<int>((x / K1) % s.R);
        const int pair = static_cast<int>(x / (static_cast<long long>(K1) * s.R));
        const int c = slot_chunk(a, pair, tok, slot);
        if (c >= 0) atomicAdd(&a.cnt[(static_cast<long long>(tok / a.qb) * pairs + pair) * a.nc + c], 1);
    }
}

// Exclusive prefix sum of the tiles per list, ceil(cnt / tile_tok), in two launches of one CTA per 1024 lists:
// segment sums first, then every CTA adds up the sums of the segments before its own and scans its segment.
// A list's first entry is its first tile x tile_tok, so the tiles of a query block cover one contiguous,
// tile-aligned range of entries.
__global__ void __launch_bounds__(1024) invert_segsum_kernel(const PArgs a) {
    __shared__ int wsum[32];
    pdl_wait();
    const int n = a.s.B * a.s.Hkv * a.nc * a.n_blocks;
    const int x = blockIdx.x * 1024 + threadIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int ct = x < n ? (a.cnt[x] + a.tile_tok - 1) / a.tile_tok : 0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ct += __shfl_xor_sync(kFullMask, ct, o);
    if (lane == 0) wsum[warp] = ct;
    __syncthreads();
    if (warp == 0) {
        int v = wsum[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFullMask, v, o);
        if (lane == 0) a.seg_tiles[blockIdx.x] = v;
    }
}

__global__ void __launch_bounds__(1024) invert_scan_kernel(const PArgs a) {
    __shared__ int wsum_t[32];
    __shared__ int wpre[32];
    pdl_wait();
    const Shape& s = a.s;
    const int per_blk = s.B * s.Hkv * a.nc;
    const int n = per_blk * a.n_blocks;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // tiles of all earlier segments
    int pre = 0;
    for (int sg = tid; sg < static_cast<int>(blockIdx.x); sg += 1024) pre += a.seg_tiles[sg];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) pre += __shfl_xor_sync(kFullMask, pre, o);
    if (lane == 0) wpre[warp] = pre;
    const int x = blockIdx.x * 1024 + tid;
    const int ce = x < n ? a.cnt[x] : 0;
    const int ct = (ce + a.tile_tok - 1) / a.tile_tok;
    int it = ct;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int nt = __shfl_up_sync(kFullMask, it, o);
        if (lane >= o) it += nt;
    }
    if (lane == 31) wsum_t[warp] = it;
    __syncthreads();
    int bt = 0;
    for (int w = 0; w < 32; ++w) bt += wpre[w] + (w < warp ? wsum_t[w] : 0);
    const int ot = bt + it - ct, oe = ot * a.tile_tok;
    if (x < n) {
        a.off[x] = oe;
        const int pair = (x % per_blk) / a.nc, c = x % a.nc;
        if (x % per_blk == 0) a.blk_toff[x / per_blk] = ot;
        for (int k = 0; k < ct; ++k)
            if (ot + k < a.max_tiles)
                a.tiles[ot + k] = make_int4(pair, c, oe + k * a.tile_tok, min(a.tile_tok, ce - k * a.tile_tok));
        if (x == n - 1) a.blk_toff[a.n_blocks] = min(ot + ct, a.max_tiles);
    }
}

// A warp takes one slot of 32 consecutive tokens: neighbouring tokens mostly hold the same chunk in a slot (the
// local window's chunks always, the selected ones whenever adjacent queries agree), so the lanes that target the
// same list are served by ONE add on its cursor: the lowest such lane reserves room for all of them.
__global__ void invert_fill_kernel(const PArgs a) {
    pdl_wait();
    const Shape& s = a.s;
    const int K1 = s.K + max_local_slots(s.W), pairs = s.B * s.Hkv;
    const int lane = threadIdx.x & 31;
    const int tblocks = (s.R + 31) / 32;
    const long long total = static_cast<long long>(pairs) * tblocks * K1;
    const long long nwarps = static_cast<long long>(gridDim.x) * (blockDim.x >> 5);
    for (long long w = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); w < total; w += nwarps) {
        const int slot = static_cast<int>(w % K1);
        const int tb = static_cast<int>((w / K1) % tblocks);
        const int pair = static_cast<int>(w / (static_cast<long long>(K1) * tblocks));
        const int tok = tb * 32 + lane;
        const int c = tok < s.R ? slot_chunk(a, pair, tok, slot) : -1;
        const long long idx = c >= 0 ? (static_cast<long long>(tok / a.qb) * pairs + pair) * a.nc + c : -1 - lane;
        const unsigned same = __match_any_sync(kFullMask, idx);
        const int leader = __ffs(same) - 1;
        int base = 0;
        if (c >= 0 && lane == leader) base = a.off[idx] + atomicAdd(&a.cursor[idx], __popc(same));
        base = __shfl_sync(kFullMask, base, leader);
        if (tok < s.R) {
            int pos = -1;
            if (c >= 0) {
                pos = base + __popc(same & ((1u << lane) - 1u));
                if (pos < a.max_tiles * a.tile_tok) a.entries[pos] = ((tok % a.qb) << 8) | slot;
            }
            a.epos[(static_cast<long long>(pair) * s.R + tok) * K1 + slot] = pos;
        }
    }
}

// ------------------------------------------------------------------------------------------ routed scores
// With a separate routing query q-hat (Eq. Q-Cal) the chunk mass of a selected slot is scale * q-hat . k'_c + b'_c,
// not the q . k'_c that the attend kernel read off its score tile: this kernel overwrites those masses.  One CTA
// per tile, one warp per entry at a time; lane l covers dimensions 4l .. 4l+3.  Local slots keep their masses.
__global__ void __launch_bounds__(128) prefill_route_scores_kernel(const PArgs a) {
    pdl_wait();
    const Shape& s = a.s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t_begin = a.blk_toff[a.blk];
    const int tile = t_begin + static_cast<int>(blockIdx.x);
    if (tile >= a.blk_toff[a.blk + 1]) return;
    const int4 rec = a.tiles[tile];
    const int pair = rec.x, c = rec.y, first = rec.z, ntok = rec.w;
    if (c >= s.C) return;
    const int b = pair / s.Hkv, gk = pair % s.Hkv, per = s.Hl / s.Hkv;
    const int e0 = a.whole ? 0 : t_begin * a.tile_tok;
    for (int ei = warp; ei < ntok; ei += 4) {
        const int e = a.entries[first + ei];
        const int tok = a.i0 + (e >> 8), slot = e & 255;
        if (slot >= s.K) continue;
#pragma unroll
        for (int h = 0; h < kG; ++h) {
            const long long lrow = (static_cast<long long>(b) * s.Hl + gk * per + (per == 1 ? 0 : h)) * s.C + c;
            const uint2 qv = *reinterpret_cast<const uint2*>(a.q + ((static_cast<long long>(b) * s.Hq + gk * kG + h) * s.R + tok) * kD + lane * 4);
            const uint2 lv = *reinterpret_cast<const uint2*>(a.lm + lrow * kD + lane * 4);
            float dotp = __uint_as_float(qv.x << 16) * __uint_as_float(lv.x << 16);
            dotp = fmaf(__uint_as_float(qv.x & 0xffff0000u), __uint_as_float(lv.x & 0xffff0000u), dotp);
            dotp = fmaf(__uint_as_float(qv.y << 16), __uint_as_float(lv.y << 16), dotp);
            dotp = fmaf(__uint_as_float(qv.y & 0xffff0000u), __uint_as_float(lv.y & 0xffff0000u), dotp);
            dotp = warp_sum(dotp);
            if (lane == 0) a.lam[static_cast<long long>(first - e0 + ei) * kG + h] = dotp * s.scale + (a.bias ? a.bias[lrow] : 0.f);
        }
    }
}

// ------------------------------------------------------------------------------------------ fuse
// One warp per (sequence, KV head, token): softmax over {surrogate scores of the selected chunks} U
// {log Z_swa} per head (Eq. HiLS weights, inter-chunk factor) and the weighted sum of the rows that
// prefill_attend wrote.  The rows are found through the entry index of every (token, slot); an entry's
// 4 heads are 1 KB contiguous (two 16-byte loads per lane); lane l covers head l/16 (and head 2 + l/16),
// elements 8*(l%16)..+7.
constexpr int kFuseWarps = 4;
constexpr int kFuseRows = 96;             // rows mixed per token: K <= 64 selected + up to 16 local chunks, 3 x 32 lanes

__global__ void __launch_bounds__(kFuseWarps * 32) prefill_fuse_kernel(const PArgs a) {
    __shared__ float wsm[kFuseWarps][kG][kFuseRows];
    __shared__ int esm[kFuseWarps][kFuseRows];
    pdl_wait();
    const Shape& s = a.s;
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int K = s.K, K1 = K + max_local_slots(s.W), nblk = a.i1 - a.i0;
    const long long total = static_cast<long long>(s.B) * s.Hkv * nblk;
    const long long w = static_cast<long long>(blockIdx.x) * kFuseWarps + wib;
    if (w >= total) return;
    const int il = static_cast<int>(w % nblk);
    const int pair = static_cast<int>(w / nblk);
    const int b = pair / s.Hkv, gk = pair % s.Hkv;
    const int tok = a.i0 + il;
    // rows to mix: the selected chunks (slots 0..nsel-1), then the chunks of the local window (slots K..K+nl-1)
    const int pos = s.pos0 + tok;                    // sequence position of this query row
    const int lc = local_lo(pos, s.W, kS) / kS;      // first local chunk = number of candidate chunks
    const int nsel = min(K, lc);
    const int nl = pos / kS - lc + 1;
    const int nrows = nsel + nl;
    const int e0 = a.whole ? 0 : a.blk_toff[a.blk] * a.tile_tok;   // first entry of this query block
    const int* ep = a.epos + (static_cast<long long>(pair) * s.R + tok) * K1;
    const float4* lam4 = reinterpret_cast<const float4*>(a.lam);
    float (*wv)[kFuseRows] = wsm[wib];
    int* ev = esm[wib];
    // entry (relative to the block) and the four heads' chunk masses of rows lane, lane + 32, lane + 64
    float lam[3][kG];
#pragma unroll
    for (int st = 0; st < 3; ++st) {
        const int r = lane + 32 * st;
        float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        if (r < nrows) {
            const int en = ep[r < nsel ? r : K + (r - nsel)] - e0;
            ev[r] = en;
            v = lam4[en];
        }
        lam[st][0] = v.x; lam[st][1] = v.y; lam[st][2] = v.z; lam[st][3] = v.w;
    }
    // the first four rows are requested before the weights are worked out (their addresses need only the entries)
    __syncwarp();
    uint4 ra[4], rb[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int r = min(u, nrows - 1);
        const __nv_bfloat16* row = a.obuf + static_cast<long long>(ev[r]) * kG * kD;
        ra[u] = obuf_load(reinterpret_cast<const uint4*>(row + lane * 8));
        rb[u] = obuf_load(reinterpret_cast<const uint4*>(row + 256 + lane * 8));
    }
    float lse_h = 0.f;
#pragma unroll
    for (int h = 0; h < kG; ++h) {
        const float Mx = warp_max(fmaxf(fmaxf(lam[0][h], lam[1][h]), lam[2][h]));
        float ex[3];
#pragma unroll
        for (int st = 0; st < 3; ++st) ex[st] = __expf(lam[st][h] - Mx);
        const float D = warp_sum(ex[0] + ex[1] + ex[2]);
        const float inv = 1.f / D;
#pragma unroll
        for (int st = 0; st < 3; ++st)
            if (lane + 32 * st < nrows) wv[h][lane + 32 * st] = ex[st] * inv;
        if (lane == h) lse_h = Mx + __logf(D);
    }
    __syncwarp();
    const int hA = lane >> 4, hB = 2 + (lane >> 4), piece = lane & 15;
    float accA[8], accB[8];
#pragma unroll
    for (int x = 0; x < 8; ++x) { accA[x] = 0.f; accB[x] = 0.f; }
    auto fma8 = [](float (&acc)[8], const uint4& raw, float wgt) {
        const uint32_t wd[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            acc[2 * x] = fmaf(wgt, __uint_as_float(wd[x] << 16), acc[2 * x]);
            acc[2 * x + 1] = fmaf(wgt, __uint_as_float(wd[x] & 0xffff0000u), acc[2 * x + 1]);
        }
    };
    // four rows at a time (8 loads in flight per lane)
    for (int r0 = 0; r0 < nrows; r0 += 4) {
        if (r0 > 0) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int r = min(r0 + u, nrows - 1);
                const __nv_bfloat16* row = a.obuf + static_cast<long long>(ev[r]) * kG * kD;
                ra[u] = obuf_load(reinterpret_cast<const uint4*>(row + lane * 8));
                rb[u] = obuf_load(reinterpret_cast<const uint4*>(row + 256 + lane * 8));
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (r0 + u < nrows) {
                fma8(accA, ra[u], wv[hA][r0 + u]);
                fma8(accB, rb[u], wv[hB][r0 + u]);
            }
        }
    }
    const long long rowA = (static_cast<long long>(b) * s.Hq + gk * kG + hA) * s.R + tok;
    const long long rowB = (static_cast<long long>(b) * s.Hq + gk * kG + hB) * s.R + tok;
    uint4 pa, pb;
    pa.x = pack_bf16(accA[0], accA[1]); pa.y = pack_bf16(accA[2], accA[3]);
    pa.z = pack_bf16(accA[4], accA[5]); pa.w = pack_bf16(accA[6], accA[7]);
    pb.x = pack_bf16(accB[0], accB[1]); pb.y = pack_bf16(accB[2], accB[3]);
    pb.z = pack_bf16(accB[4], accB[5]); pb.w = pack_bf16(accB[6], accB[7]);
    *reinterpret_cast<uint4*>(a.out + rowA * kD + piece * 8) = pa;
    *reinterpret_cast<uint4*>(a.out + rowB * kD + piece * 8) = pb;
    if (lane < kG) a.lse[(static_cast<long long>(b) * s.Hq + gk * kG + lane) * s.R + tok] = lse_h;
}

// HILS_FORCE_MMA_SELECT=1 keeps the warp-MMA selection kernel even where the tcgen05 one applies (used to
// cross-check the two implementations).
const bool g_force_mma_select = [] {
    const char* e = getenv("HILS_FORCE_MMA_SELECT");
    return e != nullptr && e[0] == '1';
}();
// HILS_PREFILL_QB overrides the query-block length (multiple of 64, for tuning runs); 0 = choose per call.
const int kQBEnv = [] {
    const char* e = getenv("HILS_PREFILL_QB");
    const int v = e ? atoi(e) : 0;
    return (v >= 64 && v % 64 == 0 && v <= (1 << 20)) ? v : 0;
}();
// Tokens per query block.  A block's tokens that selected a chunk form that chunk's list; lists of about 500 entries
// (16 tiles) amortise the chunk's K/V load and the ragged last tile, and a list holds about block * K / (visible
// chunks ~ L / 2S) entries: block ~ 4 L / K, between 4096 (the gathered Q rows of a block stay in L2) and 8192
// (16384 gains another 0.7 % on 128K tokens for twice the partial-output buffer).
int pick_query_block(const Shape& s) {
    if (kQBEnv) return kQBEnv;
    const long long want = 4ll * (static_cast<long long>(s.pos0) + s.R) / (s.K > 0 ? s.K : 1);
    int qb = kQBDefault;
    while (qb < want && qb < 2 * kQBDefault) qb *= 2;
    return qb;
}
struct Plan {
    int qb, nc, n_blocks, max_tiles, max_blk_tiles, whole;
    size_t off_cnt, off_cursor, off_ntiles, zero_bytes, off_seg, off_off, off_entries, off_epos, off_tiles, off_obuf, off_lam,
        total, obuf_tiles;
};

Plan make_plan(const Shape& s, int qb_fixed = 0) {
    Plan p;
    const size_t pairs = static_cast<size_t>(s.B) * s.Hkv;
    const int QB = qb_fixed > 0 ? qb_fixed : pick_query_block(s);
    const size_t blk = static_cast<size_t>(s.R < QB ? (s.R + kS - 1) / kS * kS : QB);
    p.qb = static_cast<int>(blk);
    const size_t nchunks = (static_cast<size_t>(s.pos0) + s.R + kS - 1) / kS;     // chunks the queries can touch
    const size_t nc = static_cast<size_t>(s.C) > nchunks ? static_cast<size_t>(s.C) : nchunks;
    p.nc = static_cast<int>(nc);
    const size_t nblocks = (static_cast<size_t>(s.R) + blk - 1) / blk;
    p.n_blocks = static_cast<int>(nblocks);
    // tiles of a block <= its entries / tile + one ragged tile per list; a block's tokens see the chunks up to its end
    const size_t tt = static_cast<size_t>(attend_tc_tile_tokens());
    size_t all_tiles = 0, max_blk = 0;
    for (size_t b = 0; b < nblocks; ++b) {
        const size_t toks = (b + 1) * blk <= static_cast<size_t>(s.R) ? blk : static_cast<size_t>(s.R) - b * blk;
        const size_t vis = ((s.pos0 + b * blk + toks) + kS - 1) / kS;
        // (and never more than its entries: a list that exists holds at least one)
        const size_t ents = pairs * toks * (s.K + max_local_slots(s.W));
        const size_t ragged = pairs * (toks * (s.K + max_local_slots(s.W)) / tt + (vis < nc ? vis : nc));
        const size_t tiles = (ents < ragged ? ents : ragged) + 1;
        all_tiles += tiles;
        max_blk = tiles > max_blk ? tiles : max_blk;
    }
    p.max_tiles = static_cast<int>(all_tiles);
    p.max_blk_tiles = static_cast<int>(max_blk);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = (off + bytes + 255) / 256 * 256; return o; };
    p.off_cnt = take(sizeof(int) * nblocks * pairs * nc);
    p.off_cursor = take(sizeof(int) * nblocks * pairs * nc);
    p.off_ntiles = take(sizeof(int) * (nblocks + 1));
    p.zero_bytes = off;                         // cnt, cursor, blk_toff are cleared together once per call
    p.off_seg = take(sizeof(int) * ((nblocks * pairs * nc + 1023) / 1024));
    p.off_off = take(sizeof(int) * nblocks * pairs * nc);
    p.off_entries = take(sizeof(int) * all_tiles * tt);
    p.off_epos = take(sizeof(int) * pairs * s.R * (s.K + max_local_slots(s.W)));
    p.off_tiles = take(sizeof(int4) * all_tiles);
    // Partial outputs of all query blocks at once while that stays under 4 GB: the fusion then runs as one launch
    // over the whole call instead of one per block (each launch pays its ramp and its last wave).
    p.whole = (nblocks > 1 && all_tiles * tt * kG * kD * sizeof(__nv_bfloat16) <= (4ull << 30)) ? 1 : 0;
    const size_t obuf_tiles = p.whole ? all_tiles : max_blk;
    p.obuf_tiles = obuf_tiles;
    p.off_obuf = take(sizeof(__nv_bfloat16) * obuf_tiles * tt * kG * kD);
    p.off_lam = take(sizeof(float) * obuf_tiles * tt * kG);
    p.total = off;
    return p;
}

}  // namespace

bool prefill_fast_supports(const Shape& s, int dtype) {
    // any window whose chunks fit the fuse kernel's row table; the warp-MMA selection fallback (K > 32) scores one
    // landmark row per KV head
    return dtype == HILS_BF16 && !s.is_decode && s.d == kD && s.S == kS && s.W >= 1 && max_local_slots(s.W) <= 16 &&
           (s.Hl == s.Hkv || (s.K <= 32 && prefill_select_tc_supports(s))) &&
           (s.Hl == s.Hkv || s.Hl == s.Hq) && s.G == kG &&
           s.K >= 1 && s.K <= 64 && static_cast<long long>(s.B) * s.Hkv * s.T < (1ll << 31) &&
           static_cast<long long>(s.B) * s.Hkv * s.C < (1ll << 24) &&
           static_cast<long long>(s.B) * s.Hkv * ((s.pos0 + s.R + kS - 1) / kS) < (1ll << 31) &&
           static_cast<long long>(s.B) * s.Hkv * s.R * (s.K + max_local_slots(s.W)) < (1ll << 31);
}

size_t prefill_fast_scratch_bytes(const Shape& s) { return make_plan(s).total; }

// The inverse index on its own (the backward pass walks the same chunk-major tiles): per-(query block, pair, chunk)
// entry lists and the tile table, built from a selection that is already in memory.
// (query blocks of kQBDefault tokens: the fp32 dq rows a block accumulates into have to stay in L2)
size_t inverse_index_bytes(const Shape& s) { return make_plan(s, kQBEnv ? kQBEnv : kQBDefault).off_obuf; }

int build_inverse_index(const Shape& s, const int32_t* sel, void* scratch, size_t bytes, InverseIndex* ix,
                        cudaStream_t stream) {
    const Plan p = make_plan(s, kQBEnv ? kQBEnv : kQBDefault);
    if (bytes < p.off_obuf) return HILS_ERR_WORKSPACE;
    const int pairs = s.B * s.Hkv;
    char* sc = static_cast<char*>(scratch);
    PArgs a = {};
    a.s = s;
    a.sel = const_cast<int32_t*>(sel);
    a.cnt = reinterpret_cast<int*>(sc + p.off_cnt);
    a.cursor = reinterpret_cast<int*>(sc + p.off_cursor);
    a.blk_toff = reinterpret_cast<int*>(sc + p.off_ntiles);
    a.n_blocks = p.n_blocks;
    a.seg_tiles = reinterpret_cast<int*>(sc + p.off_seg);
    a.off = reinterpret_cast<int*>(sc + p.off_off);
    a.entries = reinterpret_cast<int*>(sc + p.off_entries);
    a.epos = reinterpret_cast<int*>(sc + p.off_epos);
    a.tiles = reinterpret_cast<int4*>(sc + p.off_tiles);
    a.max_tiles = p.max_tiles;
    a.qb = p.qb;
    a.nc = p.nc;
    a.tile_tok = attend_tc_tile_tokens();
    if (cudaMemsetAsync(sc + p.off_cnt, 0, p.zero_bytes, stream) != cudaSuccess) return HILS_ERR_CUDA;
    const long long elems = static_cast<long long>(pairs) * s.R * (s.K + max_local_slots(s.W));
    const long long want = (elems + 255) / 256;
    const unsigned eb = static_cast<unsigned>(want < sm_count() * 16 ? want : sm_count() * 16);
    const unsigned nseg = static_cast<unsigned>((static_cast<long long>(p.n_blocks) * pairs * p.nc + 1023) / 1024);
    invert_count_kernel<<<eb, 256, 0, stream>>>(a);
    invert_segsum_kernel<<<nseg, 1024, 0, stream>>>(a);
    invert_scan_kernel<<<nseg, 1024, 0, stream>>>(a);
    invert_fill_kernel<<<eb, 256, 0, stream>>>(a);
    if (cudaGetLastError() != cudaSuccess) return HILS_ERR_CUDA;
    trace_mark("backward_invert", stream);
    ix->qb = p.qb;
    ix->nc = p.nc;
    ix->n_blocks = p.n_blocks;
    ix->max_tiles = p.max_tiles;
    ix->tile_tok = a.tile_tok;
    ix->entries = a.entries;
    ix->tiles = a.tiles;
    ix->blk_toff = a.blk_toff;
    return 4;
}

int launch_prefill_fast(const Shape& s, const Tensors& t, cudaStream_t stream) {
    const Plan p = make_plan(s);
    if (t.scratch_bytes < p.total) return HILS_ERR_WORKSPACE;
    const int pairs = s.B * s.Hkv;
    char* sc = static_cast<char*>(t.scratch);
    PArgs a;
    a.s = s;
    // PArgs::q feeds the selection fallback and the routed-score kernel: the routing query (q itself unless given)
    a.q = static_cast<const __nv_bfloat16*>(t.q_route ? t.q_route : t.q);
    a.lm = static_cast<const __nv_bfloat16*>(t.landmarks);
    a.bias = t.bias;
    a.out = static_cast<__nv_bfloat16*>(t.out);
    a.lse = t.lse;
    a.sel = t.sel_idx;
    a.status = t.status;
    a.cnt = reinterpret_cast<int*>(sc + p.off_cnt);
    a.cursor = reinterpret_cast<int*>(sc + p.off_cursor);
    a.blk_toff = reinterpret_cast<int*>(sc + p.off_ntiles);
    a.n_blocks = p.n_blocks;
    a.blk = 0;
    a.seg_tiles = reinterpret_cast<int*>(sc + p.off_seg);
    a.off = reinterpret_cast<int*>(sc + p.off_off);
    a.entries = reinterpret_cast<int*>(sc + p.off_entries);
    a.epos = reinterpret_cast<int*>(sc + p.off_epos);
    a.tiles = reinterpret_cast<int4*>(sc + p.off_tiles);
    a.obuf = reinterpret_cast<__nv_bfloat16*>(sc + p.off_obuf);
    a.lam = reinterpret_cast<float*>(sc + p.off_lam);
    a.max_tiles = p.max_tiles;
    a.qb = p.qb;
    a.nc = p.nc;
    a.tile_tok = attend_tc_tile_tokens();
    a.i0 = 0;
    a.i1 = 0;
    a.whole = p.whole;

    // K, V: boxes of 64 dims x 64 keys; partial outputs: boxes of 64 dims x 32 rows (one epilogue warp's rows)
    CUtensorMap map_k, map_v, map_lm, map_o;
    const uint64_t kv_rows = static_cast<uint64_t>(pairs) * s.T;
    if (!make_bf16_2d_map(&map_k, t.k, kv_rows, kD, 64, kS) || !make_bf16_2d_map(&map_v, t.v, kv_rows, kD, 64, kS) ||
        !make_bf16_2d_map(&map_lm, t.landmarks, static_cast<uint64_t>(pairs) * s.C, kD, 64, kS) ||
        !make_bf16_2d_map(&map_o, a.obuf, static_cast<uint64_t>(p.obuf_tiles) * a.tile_tok * kG, kD, 64, 32))
        return HILS_ERR_CUDA;

    const size_t sel_smem = kSelStages * kSelStageBytes + 64 + sizeof(unsigned long long) * 64 * (s.K + 1) + 1024;
    static PerDeviceOnce attr_once;
    if (attr_once.pending()) {
        const size_t sel_max = kSelStages * kSelStageBytes + 64 + sizeof(unsigned long long) * 64 * 65 + 1024;
        if (cudaFuncSetAttribute(prefill_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(sel_max)) != cudaSuccess)
            return HILS_ERR_CUDA;
        attr_once.done();
    }

    int launches = 0;
    const int tiles_per_seq = (s.R + kS - 1) / kS;
    // counters of the inverse index start at zero; the tcgen05 selection kernel fills the per-chunk entry counts itself
    if (cudaMemsetAsync(sc + p.off_cnt, 0, p.zero_bytes, stream) != cudaSuccess) return HILS_ERR_CUDA;
    bool counted = false;
    if (prefill_select_tc_supports(s) && !g_force_mma_select) {
        const int rc = launch_prefill_select_tc(s, a.q, t.landmarks, t.bias, t.sel_idx, t.status, a.cnt, a.qb, a.nc, stream);
        if (rc < 0) return rc;
        counted = rc == 2;
    } else {
        prefill_select_kernel<<<static_cast<unsigned>(pairs) * tiles_per_seq, 160, sel_smem, stream>>>(map_lm, a);
        if (cudaGetLastError() != cudaSuccess) return HILS_ERR_CUDA;
    }
    trace_mark("prefill_select", stream);
    ++launches;

    // inverse index for every query block at once: per-(block, pair, chunk) lists of (token, slot) entries
    // and the table of attend tiles, grouped by block
    {
        const long long elems = static_cast<long long>(pairs) * s.R * (s.K + max_local_slots(s.W));
        const long long want = (elems + 255) / 256;
        const unsigned eb = static_cast<unsigned>(want < sm_count() * 16 ? want : sm_count() * 16);
        if (!counted) {
            invert_count_kernel<<<eb, 256, 0, stream>>>(a);
            ++launches;
        }
        const unsigned nseg = static_cast<unsigned>((static_cast<long long>(p.n_blocks) * pairs * p.nc + 1023) / 1024);
        // From here on every kernel of the call is launched so that its launch and prologue overlap the previous
        // kernel's tail; each of them waits for its predecessors' results before its first dependent access.  None
        // triggers its dependents early: CTAs of the next kernel parked beside a running attend kernel cost 5 %.
        if (launch_pdl(invert_segsum_kernel, dim3(nseg), dim3(1024), 0, stream, a) != cudaSuccess ||
            launch_pdl(invert_scan_kernel, dim3(nseg), dim3(1024), 0, stream, a) != cudaSuccess ||
            launch_pdl(invert_fill_kernel, dim3(eb), dim3(256), 0, stream, a) != cudaSuccess)
            return HILS_ERR_CUDA;
        trace_mark("prefill_invert", stream);
        launches += 3;
    }
    for (int i0 = 0, blk = 0; i0 < s.R; i0 += a.qb, ++blk) {
        a.i0 = i0;
        a.i1 = s.R < i0 + a.qb ? s.R : i0 + a.qb;
        a.blk = blk;
        if (!a.whole || blk == 0) {
            // one launch per query block, or a single launch that walks all of them (whole-call output buffers)
            const CUtensorMap maps[3] = {map_k, map_v, map_o};
            const int rc = launch_prefill_attend_tc(s, t.q, maps, t.landmarks, t.bias, a.entries, a.tiles,
                                                    a.blk_toff + blk, a.lam, t.status, a.i0, a.whole,
                                                    a.whole ? p.n_blocks : 1, a.qb, stream);
            if (rc < 0) return rc;
            trace_mark("prefill_attend", stream);
            ++launches;
        }
        if (t.q_route) {
            const int ntl = (p.max_blk_tiles);
            if (launch_pdl(prefill_route_scores_kernel, dim3(static_cast<unsigned>(ntl)), dim3(128), 0, stream, a) != cudaSuccess)
                return HILS_ERR_CUDA;
            trace_mark("prefill_route_scores", stream);
            ++launches;
        }
        if (a.whole) {
            // one fusion launch after the last block's attend, over every token of the call
            if (a.i1 < s.R) continue;
            a.i0 = 0;
        }
        const long long fuse_warps = static_cast<long long>(pairs) * (a.i1 - a.i0);
        if (launch_pdl(prefill_fuse_kernel, dim3(static_cast<unsigned>((fuse_warps + kFuseWarps - 1) / kFuseWarps)),
                       dim3(kFuseWarps * 32), 0, stream, a) != cudaSuccess)
            return HILS_ERR_CUDA;
        trace_mark("prefill_fuse", stream);
        ++launches;
    }
    return launches;
}

}  // namespace hils
