// Tensor-core prefill kernels: bf16, d = 128, S = 64, G = 4, one landmark per KV head, W = 1.
//
// With independent queries the tokens that select a chunk are scattered over the sequence, so the
// path is organised CHUNK-MAJOR: K/V of a chunk are staged once and reused by every query row that
// selected it; what moves per (token, chunk) pair is the query rows in and one bf16 output row out.
//
//   prefill_select  per (sequence, KV head, 64-token tile): streams landmark tiles through a TMA ring,
//                   scores them with warp MMA for the 4 heads (Eq. surrogate top-k), takes the group
//                   max (App. C) and keeps an exact running top-K per token (ties: lower chunk id).
//   invert_*        turns sel_idx of a token block into per-chunk lists of (token, slot) entries and a
//                   table of 16-token tiles.
//   prefill_attend  persistent CTAs over the tile table: Q rows gathered as MMA A fragments, the
//                   chunk's own softmax (Eq. HiLS weights, intra-chunk factor), P V, one normalised
//                   bf16 output row and the per-head surrogate score per (token, slot).
//   prefill_fuse    per 64-token chunk: causal local attention (Eq. chunk mass) and the softmax over
//                   {surrogate scores} U {log Z_swa} that mixes the rows written by prefill_attend.
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
constexpr int kTileTok = 16;                 // tokens per attend tile (x 4 heads = 64 MMA rows)
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
    int* off;               // [pairs*C] exclusive prefix of cnt
    int* toff;              // [pairs*C] exclusive prefix of tiles per (pair, chunk)
    int* entries;           // [pairs*QB*(K+1)] (token_local << 8) | slot, grouped by (pair, chunk);
                            // slot K marks the token's own chunk (local branch)
    int4* tiles;            // [max_tiles] {pair, chunk, first entry, rows}
    __nv_bfloat16* obuf;    // [pairs*QB*(K+1)][G][128] normalised per-chunk outputs (slot K: local)
    float* lam;             // [pairs*QB][G][K+1] per-head surrogate scores; slot K: log Z_swa
    int i0, i1;             // token block [i0, i1) of the attend / fuse launch
    int blk;                // its index
    int n_blocks;           // query blocks of qb tokens
    int qb;                 // tokens per block the obuf / lam strides are sized for
    int nc;                 // chunk slots per pair in cnt/off/...: max(C, ceil(L / S))
    int tile_tok;           // entries per attend tile: 32 (tcgen05 kernel) or 16 (warp-MMA kernel)
    int max_tiles;
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
    const int ncand = ci;                       // W = 1: every earlier chunk is a candidate
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
                float u = um[v] * s.scale;
                if (bias && c < ncand) u += bias[c];
                key[v] = c < ncand ? select_key(u, c) : 0ull;
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
// Chunk attended by slot `slot` of token i0+il: a selected chunk, or (slot K) the token's own chunk.
__device__ __forceinline__ int slot_chunk(const PArgs& a, int pair, int tok, int slot) {
    if (slot == a.s.K) return tok / kS;
    return a.sel[(static_cast<long long>(pair) * a.s.R + tok) * a.s.K + slot];
}

__global__ void invert_count_kernel(const PArgs a) {
    const Shape& s = a.s;
    const int K1 = s.K + 1, pairs = s.B * s.Hkv;
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

// single CTA: exclusive prefix sums of cnt (entries) and of ceil(cnt/16) (tiles), then the tile table
__global__ void __launch_bounds__(1024) invert_scan_kernel(const PArgs a) {
    __shared__ int wsum_e[32], wsum_t[32];
    __shared__ int carry_e, carry_t;
    const Shape& s = a.s;
    const int per_blk = s.B * s.Hkv * a.nc;
    const int n = per_blk * a.n_blocks;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) { carry_e = 0; carry_t = 0; }
    __syncthreads();
    for (int base = 0; base < n; base += 1024) {
        const int x = base + tid;
        const int ce = x < n ? a.cnt[x] : 0;
        const int ct = (ce + a.tile_tok - 1) / a.tile_tok;
        int ie = ce, it = ct;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int ne = __shfl_up_sync(kFullMask, ie, o), nt = __shfl_up_sync(kFullMask, it, o);
            if (lane >= o) { ie += ne; it += nt; }
        }
        if (lane == 31) { wsum_e[warp] = ie; wsum_t[warp] = it; }
        __syncthreads();
        int be = carry_e, bt = carry_t;
        for (int w = 0; w < warp; ++w) { be += wsum_e[w]; bt += wsum_t[w]; }
        const int oe = be + ie - ce, ot = bt + it - ct;
        if (x < n) {
            a.off[x] = oe;
            a.toff[x] = ot;
            const int pair = (x % per_blk) / a.nc, c = x % a.nc;
            if (x % per_blk == 0) a.blk_toff[x / per_blk] = ot;
            for (int k = 0; k < ct; ++k)
                if (ot + k < a.max_tiles)
                    a.tiles[ot + k] = make_int4(pair, c, oe + k * a.tile_tok, min(a.tile_tok, ce - k * a.tile_tok));
        }
        __syncthreads();
        if (tid == 1023) { carry_e = oe + ce; carry_t = ot + ct; }
        __syncthreads();
    }
    if (tid == 0) a.blk_toff[a.n_blocks] = min(carry_t, a.max_tiles);
}

__global__ void invert_fill_kernel(const PArgs a) {
    const Shape& s = a.s;
    const int K1 = s.K + 1, pairs = s.B * s.Hkv;
    const long long total = static_cast<long long>(pairs) * s.R * K1;
    for (long long x = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; x < total;
         x += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int slot = static_cast<int>(x % K1);
        const int tok = static_cast<int>((x / K1) % s.R);
        const int pair = static_cast<int>(x / (static_cast<long long>(K1) * s.R));
        const int c = slot_chunk(a, pair, tok, slot);
        if (c >= 0) {
            const long long idx = (static_cast<long long>(tok / a.qb) * pairs + pair) * a.nc + c;
            const int pos = a.off[idx] + atomicAdd(&a.cursor[idx], 1);
            a.entries[pos] = ((tok % a.qb) << 8) | slot;
        }
    }
}

// ------------------------------------------------------------------------------------------ attend
// S = Q K^T for 16 rows against a 64-key tile in shared memory (two swizzled 64-dim boxes).
__device__ __forceinline__ void qk16(const uint32_t (&aq)[8][4], uint32_t ks_addr, int lane, int ntiles,
                                     float (&sc)[8][4]) {
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
        sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
        if (nt < ntiles) {
#pragma unroll
            for (int kp = 0; kp < 4; ++kp) {
                const int row = nt * 8 + (lane & 7);
                const int dim = kp * 32 + (lane >> 3) * 8;
                uint32_t r0, r1, r2, r3;
                ldmatrix_x4(ks_addr + (dim >> 6) * 8192 + swz128(row, (dim & 63) >> 3), r0, r1, r2, r3);
                mma_bf16_16816(sc[nt], aq[2 * kp], r0, r1);
                mma_bf16_16816(sc[nt], aq[2 * kp + 1], r2, r3);
            }
        }
    }
}

// O += P V for 16 rows; p[nt][0..1] row g, p[nt][2..3] row g+8; only the first `ksteps` 16-key steps.
__device__ __forceinline__ void pv16(const float (&p)[8][4], uint32_t vs_addr, int lane, int ksteps,
                                     float (&o)[16][4]) {
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
        if (kk < ksteps) {
            const uint32_t ap[4] = {pack_bf16(p[2 * kk][0], p[2 * kk][1]), pack_bf16(p[2 * kk][2], p[2 * kk][3]),
                                    pack_bf16(p[2 * kk + 1][0], p[2 * kk + 1][1]),
                                    pack_bf16(p[2 * kk + 1][2], p[2 * kk + 1][3])};
#pragma unroll
            for (int dp = 0; dp < 8; ++dp) {
                const int mat = lane >> 3;
                const int row = kk * 16 + (mat & 1) * 8 + (lane & 7);
                const int dim = dp * 16 + (mat >> 1) * 8;
                uint32_t r0, r1, r2, r3;
                ldmatrix_x4_trans(vs_addr + (dim >> 6) * 8192 + swz128(row, (dim & 63) >> 3), r0, r1, r2, r3);
                mma_bf16_16816(o[2 * dp], ap, r0, r1);
                mma_bf16_16816(o[2 * dp + 1], ap, r2, r3);
            }
        }
    }
}

__device__ __forceinline__ void load_q_frags(const __nv_bfloat16* ra, const __nv_bfloat16* rb, int t,
                                             uint32_t (&aq)[8][4]) {
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        aq[ks][0] = *reinterpret_cast<const uint32_t*>(ra + ks * 16 + 2 * t);
        aq[ks][1] = *reinterpret_cast<const uint32_t*>(rb + ks * 16 + 2 * t);
        aq[ks][2] = *reinterpret_cast<const uint32_t*>(ra + ks * 16 + 8 + 2 * t);
        aq[ks][3] = *reinterpret_cast<const uint32_t*>(rb + ks * 16 + 8 + 2 * t);
    }
}

constexpr int kStgPitch = 272;                 // bytes per staged bf16 output row (256 + 16 padding)

struct AttSmem {
    uint64_t bar;
    alignas(16) uint8_t stage[kG][16 * kStgPitch];    // read back with 16-byte loads
};

__global__ void __launch_bounds__(128, 2)
prefill_attend_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                      const PArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* kv = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* lmt = kv + 32768;                                   // 2 boxes x 8 rows x 128 B
    AttSmem& sm = *reinterpret_cast<AttSmem*>(lmt + 2048);
    const Shape& s = a.s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;
    const int K = s.K;
    const float sl2 = s.scale * kLog2e;
    const int t_begin = a.blk_toff[a.blk], n_tiles = a.blk_toff[a.blk + 1] - t_begin;
    const long long lo = t_begin + static_cast<long long>(blockIdx.x) * n_tiles / gridDim.x;
    const long long hi = t_begin + static_cast<long long>(blockIdx.x + 1) * n_tiles / gridDim.x;

    if (tid == 0) { mbar_init(&sm.bar, 1); mbar_fence_init(); }
    for (int x = tid; x < 2048 / 16; x += 128) reinterpret_cast<uint4*>(lmt)[x] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();

    int cur_pair = -1, cur_c = -1;
    uint32_t phase = 0;
    for (long long tile = lo; tile < hi; ++tile) {
        const int4 rec = a.tiles[tile];
        const int pair = rec.x, c = rec.y, first = rec.z, rows = rec.w;
        if (pair != cur_pair || c != cur_c) {
            __syncthreads();                                     // every warp is done with the old chunk
            if (tid == 0) {
                const int row = pair * s.T + c * kS;
                mbar_expect_tx(&sm.bar, 32768);
                tma_load_2d(kv, &map_k, &sm.bar, 0, row);
                tma_load_2d(kv + 8192, &map_k, &sm.bar, 64, row);
                tma_load_2d(kv + 16384, &map_v, &sm.bar, 0, row);
                tma_load_2d(kv + 24576, &map_v, &sm.bar, 64, row);
            }
            if (tid < 16) {
                // landmark of this chunk as row 0 of a 9th key tile (rows 1..7 stay zero)
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (c < s.C) v = *reinterpret_cast<const uint4*>(a.lm + (static_cast<long long>(pair) * s.C + c) * kD + tid * 8);
                *reinterpret_cast<uint4*>(lmt + (tid >> 3) * 1024 + swz128(0, tid & 7)) = v;
            }
            const bool ok = mbar_wait(&sm.bar, phase);
            phase ^= 1u;
            if (!ok) {
                if (tid == 0) set_status(a.status, kDevTimeout);
                return;
            }
            const int nv = min(kS, s.R - c * kS);
            if (nv < kS) {
                // last, partial chunk of the sequence: rows past its end may hold anything; zero the
                // V rows so that they meet their zero probabilities safely
                for (int x = tid; x < (kS - nv) * 16; x += 128) {
                    const int row = nv + (x >> 4), piece = x & 15;
                    *reinterpret_cast<uint4*>(kv + 16384 + (piece >> 3) * 8192 + swz128(row, piece & 7)) = make_uint4(0u, 0u, 0u, 0u);
                }
            }
            __syncthreads();
            cur_pair = pair;
            cur_c = c;
        }
        const int b = pair / s.Hkv, gk = pair % s.Hkv;
        const int eA = a.entries[first + min(g, rows - 1)], eB = a.entries[first + min(g + 8, rows - 1)];
        const int ilA = eA >> 8, ilB = eB >> 8;
        const __nv_bfloat16* qh = a.q + (static_cast<long long>(b) * s.Hq + gk * kG + warp) * s.R * kD;
        uint32_t aq[8][4];
        load_q_frags(qh + static_cast<long long>(a.i0 + ilA) * kD, qh + static_cast<long long>(a.i0 + ilB) * kD, t, aq);

        const uint32_t ks_addr = smem_u32(kv), vs_addr = ks_addr + 16384;
        float sc[8][4];
        qk16(aq, ks_addr, lane, 8, sc);
        // surrogate score of this chunk for the row's head: q . landmark (column 0 of the 9th tile)
        float sl[4] = {0.f, 0.f, 0.f, 0.f};
        {
            const uint32_t la = smem_u32(lmt);
#pragma unroll
            for (int kp = 0; kp < 4; ++kp) {
                const int dim = kp * 32 + (lane >> 3) * 8;
                uint32_t r0, r1, r2, r3;
                ldmatrix_x4(la + (dim >> 6) * 1024 + swz128(lane & 7, (dim & 63) >> 3), r0, r1, r2, r3);
                mma_bf16_16816(sl, aq[2 * kp], r0, r1);
                mma_bf16_16816(sl, aq[2 * kp + 1], r2, r3);
            }
        }
        // rows of the chunk's own tokens (slot K) are the local branch: causal inside the chunk
        const bool locA = (eA & 255) == K, locB = (eB & 255) == K;
        const int limA = locA ? a.i0 + ilA - c * kS : kS - 1, limB = locB ? a.i0 + ilB - c * kS : kS - 1;
        float mA = -INFINITY, mB = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const int key = nt * 8 + 2 * t;
            if (key > limA) sc[nt][0] = -INFINITY;
            if (key + 1 > limA) sc[nt][1] = -INFINITY;
            if (key > limB) sc[nt][2] = -INFINITY;
            if (key + 1 > limB) sc[nt][3] = -INFINITY;
            mA = fmaxf(mA, fmaxf(sc[nt][0], sc[nt][1]));
            mB = fmaxf(mB, fmaxf(sc[nt][2], sc[nt][3]));
        }
        mA = fmaxf(mA, __shfl_xor_sync(kFullMask, mA, 1)); mA = fmaxf(mA, __shfl_xor_sync(kFullMask, mA, 2));
        mB = fmaxf(mB, __shfl_xor_sync(kFullMask, mB, 1)); mB = fmaxf(mB, __shfl_xor_sync(kFullMask, mB, 2));
        float zA = 0.f, zB = 0.f;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            sc[nt][0] = exp2f((sc[nt][0] - mA) * sl2); sc[nt][1] = exp2f((sc[nt][1] - mA) * sl2);
            sc[nt][2] = exp2f((sc[nt][2] - mB) * sl2); sc[nt][3] = exp2f((sc[nt][3] - mB) * sl2);
            zA += sc[nt][0] + sc[nt][1];
            zB += sc[nt][2] + sc[nt][3];
        }
        zA += __shfl_xor_sync(kFullMask, zA, 1); zA += __shfl_xor_sync(kFullMask, zA, 2);
        zB += __shfl_xor_sync(kFullMask, zB, 1); zB += __shfl_xor_sync(kFullMask, zB, 2);
        float o[16][4];
#pragma unroll
        for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
        pv16(sc, vs_addr, lane, 4, o);
        const float iA = 1.f / zA, iB = 1.f / zB;
        uint8_t* stg = sm.stage[warp];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            *reinterpret_cast<uint32_t*>(stg + g * kStgPitch + (i * 8 + 2 * t) * 2) = pack_bf16(o[i][0] * iA, o[i][1] * iA);
            *reinterpret_cast<uint32_t*>(stg + (g + 8) * kStgPitch + (i * 8 + 2 * t) * 2) = pack_bf16(o[i][2] * iB, o[i][3] * iB);
        }
        if (t == 0) {
            const float bb = (a.bias && c < s.C) ? a.bias[static_cast<long long>(pair) * s.C + c] : 0.f;
            // mass of the row's chunk: the surrogate score, or log Z_swa for the local branch
            if (g < rows)
                a.lam[((static_cast<long long>(pair) * a.qb + ilA) * kG + warp) * (K + 1) + (eA & 255)] =
                    locA ? mA * s.scale + __logf(zA) : sl[0] * s.scale + bb;
            if (g + 8 < rows)
                a.lam[((static_cast<long long>(pair) * a.qb + ilB) * kG + warp) * (K + 1) + (eB & 255)] =
                    locB ? mB * s.scale + __logf(zB) : sl[2] * s.scale + bb;
        }
        __syncwarp();
        // coalesced 256-byte rows: 16 lanes x 16 B per row, two rows per instruction
#pragma unroll
        for (int rr = 0; rr < 8; ++rr) {
            const int row = rr * 2 + (lane >> 4), piece = lane & 15;
            if (row < rows) {
                const int e = a.entries[first + row];
                const uint4 v = *reinterpret_cast<const uint4*>(stg + row * kStgPitch + piece * 16);
                __nv_bfloat16* dst = a.obuf + (((static_cast<long long>(pair) * a.qb + (e >> 8)) * (K + 1) + (e & 255)) * kG + warp) * kD;
                *reinterpret_cast<uint4*>(dst + piece * 8) = v;
            }
        }
        __syncwarp();
    }
}

// ------------------------------------------------------------------------------------------ fuse
// One warp per (sequence, KV head, token): softmax over {surrogate scores of the selected chunks} U
// {log Z_swa} per head (Eq. HiLS weights, inter-chunk factor) and the weighted sum of the rows that
// prefill_attend wrote.  Pure streaming: a slot's 4 heads are 1 KB contiguous (two 16-byte loads per
// lane); lane l covers head l/16 (and head 2 + l/16), elements 8*(l%16)..+7.
constexpr int kFuseWarps = 8;

__global__ void __launch_bounds__(kFuseWarps * 32) prefill_fuse_kernel(const PArgs a) {
    __shared__ float wsm[kFuseWarps][kG][68];
    const Shape& s = a.s;
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int K = s.K, K1 = K + 1, nblk = a.i1 - a.i0;
    const long long total = static_cast<long long>(s.B) * s.Hkv * nblk;
    const long long w = static_cast<long long>(blockIdx.x) * kFuseWarps + wib;
    if (w >= total) return;
    const int il = static_cast<int>(w % nblk);
    const int pair = static_cast<int>(w / nblk);
    const int b = pair / s.Hkv, gk = pair % s.Hkv;
    const int tok = a.i0 + il;
    const int nsel = min(K, tok / kS);               // W = 1: a token of chunk ci has ci candidates
    const float* lrow = a.lam + (static_cast<long long>(pair) * a.qb + il) * kG * K1;
    float (*wv)[68] = wsm[wib];
    float lse_h = 0.f;
#pragma unroll
    for (int h = 0; h < kG; ++h) {
        const float l0 = lane < nsel ? lrow[h * K1 + lane] : -INFINITY;
        const float l1 = lane + 32 < nsel ? lrow[h * K1 + lane + 32] : -INFINITY;
        const float ll = lrow[h * K1 + K];
        const float Mx = warp_max(fmaxf(fmaxf(l0, l1), ll));
        const float e0 = __expf(l0 - Mx), e1 = __expf(l1 - Mx), el = __expf(ll - Mx);
        const float D = warp_sum(e0 + e1) + el;
        const float inv = 1.f / D;
        if (lane < nsel) wv[h][lane] = e0 * inv;
        if (lane + 32 < nsel) wv[h][lane + 32] = e1 * inv;
        if (lane == 0) wv[h][64] = el * inv;
        if (lane == h) lse_h = Mx + __logf(D);
    }
    __syncwarp();
    const int hA = lane >> 4, hB = 2 + (lane >> 4), piece = lane & 15;
    const __nv_bfloat16* ob = a.obuf + (static_cast<long long>(pair) * a.qb + il) * K1 * kG * kD;
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
    // local slot first, then the selected slots four at a time (8 loads in flight per lane)
    {
        const __nv_bfloat16* row = ob + static_cast<long long>(K) * kG * kD;
        const uint4 ra = obuf_load(reinterpret_cast<const uint4*>(row + lane * 8));
        const uint4 rb = obuf_load(reinterpret_cast<const uint4*>(row + 256 + lane * 8));
        fma8(accA, ra, wv[hA][64]);
        fma8(accB, rb, wv[hB][64]);
    }
    for (int sl0 = 0; sl0 < nsel; sl0 += 4) {
        uint4 ra[4], rb[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int sl = min(sl0 + u, nsel - 1);
            const __nv_bfloat16* row = ob + static_cast<long long>(sl) * kG * kD;
            ra[u] = obuf_load(reinterpret_cast<const uint4*>(row + lane * 8));
            rb[u] = obuf_load(reinterpret_cast<const uint4*>(row + 256 + lane * 8));
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (sl0 + u < nsel) {
                fma8(accA, ra[u], wv[hA][sl0 + u]);
                fma8(accB, rb[u], wv[hB][sl0 + u]);
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

// HILS_FORCE_MMA_SELECT=1 / HILS_FORCE_MMA_ATTEND=1 keep the warp-MMA kernels even where the tcgen05
// ones apply (used to cross-check the two implementations).
const bool g_force_mma_select = [] {
    const char* e = getenv("HILS_FORCE_MMA_SELECT");
    return e != nullptr && e[0] == '1';
}();
// HILS_PREFILL_QB overrides the query-block length (multiple of 64, for tuning runs).
const int kQB = [] {
    const char* e = getenv("HILS_PREFILL_QB");
    const int v = e ? atoi(e) : 0;
    return (v >= 64 && v % 64 == 0 && v <= (1 << 20)) ? v : kQBDefault;
}();
const bool g_force_mma_attend = [] {
    const char* e = getenv("HILS_FORCE_MMA_ATTEND");
    return e != nullptr && e[0] == '1';
}();

struct Plan {
    int qb, nc, n_blocks, max_tiles;
    size_t off_cnt, off_cursor, off_ntiles, zero_bytes, off_off, off_toff, off_entries, off_tiles, off_obuf, off_lam,
        total;
};

Plan make_plan(const Shape& s) {
    Plan p;
    const size_t pairs = static_cast<size_t>(s.B) * s.Hkv;
    const size_t blk = static_cast<size_t>(s.R < kQB ? (s.R + kS - 1) / kS * kS : kQB);
    p.qb = static_cast<int>(blk);
    const size_t nc = static_cast<size_t>(s.C > (s.R + kS - 1) / kS ? s.C : (s.R + kS - 1) / kS);
    p.nc = static_cast<int>(nc);
    const size_t nblocks = (static_cast<size_t>(s.R) + blk - 1) / blk;
    p.n_blocks = static_cast<int>(nblocks);
    p.max_tiles = static_cast<int>(pairs * s.R * (s.K + 1) / kTileTok + nblocks * pairs * nc);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = (off + bytes + 255) / 256 * 256; return o; };
    p.off_cnt = take(sizeof(int) * nblocks * pairs * nc);
    p.off_cursor = take(sizeof(int) * nblocks * pairs * nc);
    p.off_ntiles = take(sizeof(int) * (nblocks + 1));
    p.zero_bytes = off;                         // cnt, cursor, blk_toff are cleared together once per call
    p.off_off = take(sizeof(int) * nblocks * pairs * nc);
    p.off_toff = take(sizeof(int) * nblocks * pairs * nc);
    p.off_entries = take(sizeof(int) * pairs * s.R * (s.K + 1));
    p.off_tiles = take(sizeof(int4) * static_cast<size_t>(p.max_tiles));
    p.off_obuf = take(sizeof(__nv_bfloat16) * pairs * blk * (s.K + 1) * kG * kD);
    p.off_lam = take(sizeof(float) * pairs * blk * kG * (s.K + 1));
    p.total = off;
    return p;
}

}  // namespace

bool prefill_fast_supports(const Shape& s, int dtype) {
    return dtype == HILS_BF16 && !s.is_decode && s.d == kD && s.S == kS && s.W == 1 && s.Hl == s.Hkv && s.G == kG &&
           s.K >= 1 && s.K <= 64 && static_cast<long long>(s.B) * s.Hkv * s.T < (1ll << 31) &&
           static_cast<long long>(s.B) * s.Hkv * s.C < (1ll << 24) &&
           static_cast<long long>(s.B) * s.Hkv * ((s.R + kS - 1) / kS) < (1ll << 31) &&
           static_cast<long long>(s.B) * s.Hkv * s.R * (s.K + 1) < (1ll << 31);
}

size_t prefill_fast_scratch_bytes(const Shape& s) { return make_plan(s).total; }

int launch_prefill_fast(const Shape& s, const Tensors& t, cudaStream_t stream) {
    const Plan p = make_plan(s);
    if (t.scratch_bytes < p.total) return HILS_ERR_WORKSPACE;
    const int pairs = s.B * s.Hkv;
    char* sc = static_cast<char*>(t.scratch);
    PArgs a;
    a.s = s;
    a.q = static_cast<const __nv_bfloat16*>(t.q);
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
    a.off = reinterpret_cast<int*>(sc + p.off_off);
    a.toff = reinterpret_cast<int*>(sc + p.off_toff);
    a.entries = reinterpret_cast<int*>(sc + p.off_entries);
    a.tiles = reinterpret_cast<int4*>(sc + p.off_tiles);
    a.obuf = reinterpret_cast<__nv_bfloat16*>(sc + p.off_obuf);
    a.lam = reinterpret_cast<float*>(sc + p.off_lam);
    a.max_tiles = p.max_tiles;
    a.qb = p.qb;
    a.nc = p.nc;
    a.tile_tok = g_force_mma_attend ? kTileTok : attend_tc_tile_tokens();
    a.i0 = 0;
    a.i1 = 0;

    CUtensorMap map_k, map_v, map_lm;
    const uint64_t kv_rows = static_cast<uint64_t>(pairs) * s.T;
    if (!make_bf16_2d_map(&map_k, t.k, kv_rows, kD, 64, kS) || !make_bf16_2d_map(&map_v, t.v, kv_rows, kD, 64, kS) ||
        !make_bf16_2d_map(&map_lm, t.landmarks, static_cast<uint64_t>(pairs) * s.C, kD, 64, kS))
        return HILS_ERR_CUDA;

    const size_t sel_smem = kSelStages * kSelStageBytes + 64 + sizeof(unsigned long long) * 64 * (s.K + 1) + 1024;
    const size_t att_smem = 32768 + 2048 + sizeof(AttSmem) + 1024;
    static bool attr_done = false;
    if (!attr_done) {
        const size_t sel_max = kSelStages * kSelStageBytes + 64 + sizeof(unsigned long long) * 64 * 65 + 1024;
        if (cudaFuncSetAttribute(prefill_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(sel_max)) != cudaSuccess ||
            cudaFuncSetAttribute(prefill_attend_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(att_smem)) != cudaSuccess)
            return HILS_ERR_CUDA;
        attr_done = true;
    }

    int launches = 0;
    const int tiles_per_seq = (s.R + kS - 1) / kS;
    if (prefill_select_tc_supports(s) && !g_force_mma_select) {
        const int rc = launch_prefill_select_tc(s, t.q, t.landmarks, t.bias, t.sel_idx, t.status, stream);
        if (rc < 0) return rc;
    } else {
        prefill_select_kernel<<<static_cast<unsigned>(pairs) * tiles_per_seq, 160, sel_smem, stream>>>(map_lm, a);
        if (cudaGetLastError() != cudaSuccess) return HILS_ERR_CUDA;
    }
    trace_mark("prefill_select", stream);
    ++launches;

    // inverse index for every query block at once: per-(block, pair, chunk) lists of (token, slot) entries
    // and the table of attend tiles, grouped by block
    if (cudaMemsetAsync(sc + p.off_cnt, 0, p.zero_bytes, stream) != cudaSuccess) return HILS_ERR_CUDA;
    {
        const long long elems = static_cast<long long>(pairs) * s.R * (s.K + 1);
        const long long want = (elems + 255) / 256;
        const unsigned eb = static_cast<unsigned>(want < 148 * 16 ? want : 148 * 16);
        invert_count_kernel<<<eb, 256, 0, stream>>>(a);
        invert_scan_kernel<<<1, 1024, 0, stream>>>(a);
        invert_fill_kernel<<<eb, 256, 0, stream>>>(a);
        if (cudaGetLastError() != cudaSuccess) return HILS_ERR_CUDA;
        trace_mark("prefill_invert", stream);
        launches += 3;
    }
    for (int i0 = 0, blk = 0; i0 < s.R; i0 += a.qb, ++blk) {
        a.i0 = i0;
        a.i1 = s.R < i0 + a.qb ? s.R : i0 + a.qb;
        a.blk = blk;
        const int nblk = a.i1 - a.i0;
        if (g_force_mma_attend) {
            prefill_attend_kernel<<<148 * 2, 128, att_smem, stream>>>(map_k, map_v, a);
            if (cudaGetLastError() != cudaSuccess) return HILS_ERR_CUDA;
        } else {
            const CUtensorMap maps_kv[2] = {map_k, map_v};
            const int rc = launch_prefill_attend_tc(s, t.q, maps_kv, t.landmarks, t.bias, a.entries, a.tiles,
                                                    a.blk_toff + blk, a.obuf, a.lam, t.status, a.i0, a.qb, stream);
            if (rc < 0) return rc;
        }
        trace_mark("prefill_attend", stream);
        const long long fuse_warps = static_cast<long long>(pairs) * nblk;
        prefill_fuse_kernel<<<static_cast<unsigned>((fuse_warps + kFuseWarps - 1) / kFuseWarps), kFuseWarps * 32, 0, stream>>>(a);
        if (cudaGetLastError() != cudaSuccess) return HILS_ERR_CUDA;
        trace_mark("prefill_fuse", stream);
        launches += 2;
    }
    return launches;
}

}  // namespace hils
