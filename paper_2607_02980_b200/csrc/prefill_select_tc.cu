// Landmark scoring + exact top-K for prefill on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// One persistent CTA per SM walks (sequence, KV head, 128-token tile) triples, heavy tiles first; the next tile's
// queries and first scores are fetched and computed while the epilogue finishes the previous tile.  The tile's queries (4 heads x 128 tokens x 128 d)
// stay in shared memory; landmark tiles of 64 chunks stream through a TMA ring.  One thread issues
// tcgen05.mma (M = 128 tokens, N = 64 chunks, K = 128) once per head into tensor memory, double
// buffered; the four epilogue warps own one token per thread (token = TMEM lane), read the four
// heads' scores, take the group max (App. C) and keep the token's exact running top-K
// (Eq. surrogate top-k; equal scores go to the lower chunk id).  A token's candidates that beat its current
// K-th best score are appended, in arrival order = ascending chunk id, to its pool in shared memory; the N best
// SCORES so far stay sorted in registers.  When a pool of the warp may fill up, every thread sorts the scores
// appended since the last time (register bitonic network on 32-bit values: one max and one min per
// compare-exchange), merges them into its sorted list, reads the new K-th best score off it and filters its pool
// in place: everything above that score and the earliest of those equal to it, exactly K entries, still in
// ascending chunk order -- which is the order the selection is written in.  The number of such compactions grows
// with log(candidates / K), not with the candidates.
#include "internal.h"
#include "tma.cuh"

namespace hils {
namespace {

constexpr int kD = 128;
constexpr int kS = 64;
constexpr int kG = 4;
constexpr int kTileTok = 128;
constexpr int kLmStages = 2;
constexpr int kLmStageBytes = kS * kD * 2;          // 64 landmark rows = two 8 KB K-blocks
constexpr int kQBytes = kG * kTileTok * kD * 2;     // 128 KB
constexpr int kMaxK = 32;
constexpr int kRoom = 32;                           // candidates a pool takes between two compactions
constexpr int kThreads = 192;                       // 4 epilogue warps, 1 TMA warp, 1 MMA warp
constexpr uint32_t kTmemCols = 512;                 // 2 buffers x 4 heads x 64 columns

struct TcArgs {
    Shape s;
    const float* bias;
    int32_t* sel;
    int* status;
    // optional: per-(query block, pair, chunk) counts of the (token, slot) entries that attend each chunk -- the
    // first step of the inverse index, taken here because the selections are at hand (NULL: not wanted)
    int* cnt;
    int qb, nc;        // tokens per query block (a multiple of the 128-token tile), chunk slots per pair in cnt
};

struct TcSmem {
    uint64_t q_empty;          // every MMA of the tile has completed: its query tile may be overwritten
    uint64_t q_full;
    uint64_t full[kLmStages];
    uint64_t empty[kLmStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    int abort;                 // a bounded wait of an epilogue thread ran out: every epilogue warp leaves after the tile
};

// Sorts N scores in registers, largest first (bitonic network, fully unrolled: static register indices; a
// compare-exchange is one max and one min).
template <int N>
__device__ __forceinline__ void bitonic_sort_desc(float (&a)[N]) {
    constexpr int kLog = N == 32 ? 5 : 4;
#pragma unroll
    for (int ks = 1; ks <= kLog; ++ks) {
#pragma unroll
        for (int js = kLog - 1; js >= 0; --js) {
            if (js >= ks) continue;
            const int k = 1 << ks, j = 1 << js;
#pragma unroll
            for (int i = 0; i < N; ++i) {
                const int l = i ^ j;
                if (l > i) {
                    const bool desc = (i & k) == 0;
                    const float hi = fmaxf(a[i], a[l]), lo = fminf(a[i], a[l]);
                    a[i] = desc ? hi : lo;
                    a[l] = desc ? lo : hi;
                }
            }
        }
    }
}
// Sorts a bitonic sequence of N scores, largest first.
template <int N>
__device__ __forceinline__ void bitonic_merge_desc(float (&a)[N]) {
    constexpr int kLog = N == 32 ? 5 : 4;
#pragma unroll
    for (int js = kLog - 1; js >= 0; --js) {
        const int j = 1 << js;
#pragma unroll
        for (int i = 0; i < N; ++i) {
            const int l = i ^ j;
            if (l > i) {
                const float hi = fmaxf(a[i], a[l]), lo = fminf(a[i], a[l]);
                a[i] = hi;
                a[l] = lo;
            }
        }
    }
}

// N = length of the per-token sorted score list: 16 for K <= 16, else 32; a pool has room for kRoom = 32 candidates
// appended between two compactions (fewer, larger compactions are cheaper than more, smaller ones).
// PERHEAD: one landmark row (and bias) per query head (App. C) instead of one per KV head.  A template parameter, not
// a run-time branch: the scan loop's code has to stay small (the kernel is sensitive to instruction fetch).
template <int N, bool PERHEAD>
__global__ void __launch_bounds__(kThreads, 1)
prefill_select_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_lm,
                         const TcArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* qs = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* lms = qs + kQBytes;
    unsigned long long* lists = reinterpret_cast<unsigned long long*>(lms + kLmStages * kLmStageBytes);   // [2 kMaxK][128]
    TcSmem& sm = *reinterpret_cast<TcSmem*>(lists + 2 * kMaxK * kTileTok);

    const Shape& s = a.s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int pairs = s.B * s.Hkv;
    const int tiles_per_seq = (s.R + kTileTok - 1) / kTileTok;
    const int n_tiles = pairs * tiles_per_seq;
    const int K = s.K;
    constexpr int per = PERHEAD ? kG : 1;     // landmark rows per chunk
    // A CTA walks the tiles blockIdx.x, blockIdx.x + gridDim.x, ... (heavy tiles first): the query tile and the first
    // scores of the next tile are fetched and computed while the epilogue still finishes the previous one.  Every
    // role derives the same tile sequence; tiles without candidates touch no barrier.
    auto tile_of = [&](int idx, int& ti, int& pair, int& nsteps) {
        ti = tiles_per_seq - 1 - idx / pairs;
        pair = idx % pairs;
        // candidates of a token = the chunks left of its local window (Sec. 2.1); the tile's last token has the most
        const int last_tok = min(s.R, (ti + 1) * kTileTok) - 1;
        const int ncand_max = local_lo(s.pos0 + last_tok, s.W, kS) / kS;
        nsteps = (ncand_max + kS - 1) / kS;
    };

    if (tid == 0) {
        mbar_init(&sm.q_full, 1);
        mbar_init(&sm.q_empty, 1);
        sm.abort = 0;
        for (int i = 0; i < kLmStages; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&sm.tmem_full[i], 1); mbar_init(&sm.tmem_empty[i], 4); }
        mbar_fence_init();
        tma_prefetch_desc(&map_q);
        tma_prefetch_desc(&map_lm);
    }
    if (warp == 5) tmem_alloc(&sm.tmem_base, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = sm.tmem_base;

    if (warp == 4) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t n_lm = 0;            // landmark tiles requested so far, over all tiles of this CTA
            int tn = 0;                   // tiles with candidates so far
            bool ok = true;
            for (int idx = blockIdx.x; idx < n_tiles && ok; idx += gridDim.x) {
                int ti, pair, nsteps;
                tile_of(idx, ti, pair, nsteps);
                if (nsteps == 0) continue;
                const int b = pair / s.Hkv, gk = pair % s.Hkv;
                if (tn > 0) ok = mbar_wait(&sm.q_empty, (tn - 1) & 1);
                if (!ok) break;
                mbar_expect_tx(&sm.q_full, kQBytes);
                for (int h = 0; h < kG; ++h) {
                    const int row = (b * s.Hq + gk * kG + h) * s.R + ti * kTileTok;
                    tma_load_2d(qs + h * 32768, &map_q, &sm.q_full, 0, row);
                    tma_load_2d(qs + h * 32768 + 16384, &map_q, &sm.q_full, 64, row);
                }
                // landmark tiles in ring order: step it, landmark head hh (per = 1: one tile per step for all heads;
                // per = G: one tile per query head, App. C)
                const int ntiles = nsteps * per;
                for (int n = 0; n < ntiles && ok; ++n, ++n_lm) {
                    const int st = n_lm % kLmStages, it = n / per, hh = n % per;
                    if (n_lm >= kLmStages) ok = mbar_wait(&sm.empty[st], ((n_lm / kLmStages) - 1) & 1);
                    if (!ok) break;
                    uint8_t* dst = lms + st * kLmStageBytes;
                    const int row = ((b * s.Hl + gk * per + hh)) * s.C + it * kS;
                    mbar_expect_tx(&sm.full[st], kLmStageBytes);
                    tma_load_2d(dst, &map_lm, &sm.full[st], 0, row);
                    tma_load_2d(dst + 8192, &map_lm, &sm.full[st], 64, row);
                }
                ++tn;
            }
            if (!ok) set_status(a.status, kDevTimeout);
            // own copies in flight: the last query tile and the last stages must have landed before exit
            if (tn > 0) mbar_wait(&sm.q_full, (tn - 1) & 1);
            for (uint32_t n = n_lm > kLmStages ? n_lm - kLmStages : 0; n < n_lm; ++n)
                mbar_wait(&sm.full[n % kLmStages], (n / kLmStages) & 1);
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(kTileTok, kS);
            // S_h = Q_h x landmark tile^T (M = 128 tokens, N = 64 chunks, K = 128) into head h's 64 columns
            auto issue_head = [&](uint32_t d_tmem, uint32_t q_addr, uint32_t lm_addr) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t da = umma_desc_k128(q_addr + (ks >> 2) * 16384 + (ks & 3) * 32);
                    const uint64_t db = umma_desc_k128(lm_addr + (ks >> 2) * 8192 + (ks & 3) * 32);
                    umma_bf16(d_tmem, da, db, idesc, ks > 0 ? 1u : 0u);
                }
            };
            const uint32_t q0 = smem_u32(qs);
            uint32_t n_lm = 0, n_step = 0;     // landmark tiles / steps so far, over all tiles of this CTA
            int tn = 0;
            bool ok = true;
            for (int idx = blockIdx.x; idx < n_tiles && ok; idx += gridDim.x) {
                int ti, pair, nsteps;
                tile_of(idx, ti, pair, nsteps);
                if (nsteps == 0) continue;
                ok = mbar_wait(&sm.q_full, tn & 1);
                for (int it = 0; it < nsteps && ok; ++it, ++n_step) {
                    const uint32_t buf = n_step & 1u;
                    if (n_step >= 2) ok = mbar_wait(&sm.tmem_empty[buf], ((n_step >> 1) - 1) & 1);
                    if (!ok) break;
                    if (per == 1) {
                        // one landmark tile for the four query heads
                        const uint32_t st = n_lm % kLmStages;
                        ok = mbar_wait(&sm.full[st], (n_lm / kLmStages) & 1);
                        if (!ok) break;
                        tc_fence_after_sync();
                        const uint32_t lm_addr = smem_u32(lms + st * kLmStageBytes);
#pragma unroll
                        for (int h = 0; h < kG; ++h) issue_head(tmem_base + buf * 256 + h * kS, q0 + h * 32768, lm_addr);
                        umma_commit(&sm.empty[st]);        // landmark stage reusable once these MMAs are done
                        ++n_lm;
                    } else {
                        // one landmark tile per query head (App. C), in ring order
#pragma unroll
                        for (int h = 0; h < kG; ++h) {
                            const uint32_t st = n_lm % kLmStages;
                            if (ok) ok = mbar_wait(&sm.full[st], (n_lm / kLmStages) & 1);
                            if (ok) {
                                tc_fence_after_sync();
                                issue_head(tmem_base + buf * 256 + h * kS, q0 + h * 32768, smem_u32(lms + st * kLmStageBytes));
                                umma_commit(&sm.empty[st]);
                                ++n_lm;
                            }
                        }
                        if (!ok) break;
                    }
                    umma_commit(&sm.tmem_full[buf]);       // scores of this step readable
                }
                if (ok) umma_commit(&sm.q_empty);          // the query tile may be replaced once all of these are done
                ++tn;
            }
            if (!ok) set_status(a.status, kDevTimeout);
        }
    } else {
        // ------------------------------------------------------------------ epilogue: one token per thread
        const int row = warp * 32 + lane;
        const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
        uint32_t n_step = 0;               // steps so far, over all tiles of this CTA
        bool ok = true;
        for (int idx = blockIdx.x; idx < n_tiles; idx += gridDim.x) {
        int ti, pair, nsteps;
        tile_of(idx, ti, pair, nsteps);
        const int b = pair / s.Hkv, gk = pair % s.Hkv;
        const int tok = ti * kTileTok + row;
        const int my_ncand = local_lo(s.pos0 + tok, s.W, kS) / kS;
        // The token's pool of raw (score bits, chunk id) pairs in arrival order = ascending chunk id: entry e at
        // pool[e * 128]; the first `kept` entries survived the last compaction (at most K), the rest were appended
        // since (at most kRoom).
        unsigned long long* pool = lists + tid;
        // bias rows of this KV head's landmark heads (per = 1: one row, shared by the four query heads)
        const float* bias = a.bias ? a.bias + (static_cast<long long>(b) * s.Hl + gk * per) * s.C : nullptr;
        float tau_f = -INFINITY;           // score of the K-th best candidate so far: the filter of the scan
        float best[N];                     // the N best scores so far, largest first (-inf = none)
#pragma unroll
        for (int e = 0; e < N; ++e) best[e] = -INFINITY;
        int cnt = 0, kept = 0;

        for (int it = 0; it < nsteps && ok; ++it, ++n_step) {
            const uint32_t buf = n_step & 1u;
            ok = mbar_wait(&sm.tmem_full[buf], (n_step >> 1) & 1);
            if (!ok) break;
            tc_fence_after_sync();
            const bool tail = (it + 1) * kS > my_ncand;     // only the last step holds chunks this token may not see
            // 8 candidates per round (a short loop body: the code has to stay resident close to the core); the group
            // scores of 16 candidates are read from tensor memory and reduced over the heads every other round
            float u16[16];
#pragma unroll 1
            for (int cb = 0; cb < 8; ++cb) {
                if ((cb & 1) == 0) {
                    float r[4][16];
                    const uint32_t col = t_lane + buf * 256 + cb * 8;
                    tmem_ld16x4(col, col + kS, col + 2 * kS, col + 3 * kS, r);
                    const int cbase = it * kS + cb * 8;
                    if (PERHEAD && bias != nullptr) {
                        // every head adds its own bias before the maximum over the group (App. C)
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int cc = min(cbase + j, s.C - 1);
                            u16[j] = fmaxf(fmaxf(fmaf(r[0][j], s.scale, bias[cc]), fmaf(r[1][j], s.scale, bias[s.C + cc])),
                                           fmaxf(fmaf(r[2][j], s.scale, bias[2 * s.C + cc]), fmaf(r[3][j], s.scale, bias[3 * s.C + cc]))) + 0.0f;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            float u = fmaxf(fmaxf(r[0][j], r[1][j]), fmaxf(r[2][j], r[3][j])) * s.scale;
                            if (bias) u += bias[min(cbase + j, s.C - 1)];
                            u16[j] = u + 0.0f;                 // -0 folds into +0: scores compare as numbers
                        }
                    }
                }
                const int c0 = it * kS + cb * 8;
                // Filter on the score: a candidate that only EQUALS the K-th best score so far loses to the K
                // candidates at or above it, which all have lower chunk ids.  Branch-free append: the slot is
                // written always and kept only when the candidate passes.
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float u = (cb & 1) ? u16[8 + j] : u16[j];
                    const int c = c0 + j;
                    const bool pass = u > tau_f && (!tail || c < my_ncand);
                    pool[cnt * kTileTok] = (static_cast<unsigned long long>(__float_as_uint(u)) << 32) | static_cast<uint32_t>(c);
                    cnt += pass ? 1 : 0;
                }
                // Compaction (one call site: the code is large): when a row of the warp may overflow on the next
                // round (at most 8 appends between checks), and once after the last round.
                const bool last_round = it + 1 == nsteps && cb == 7;
                if (__any_sync(kFullMask, cnt - kept > kRoom - 8) || last_round) {
                    // the N best scores of (best so far) + (appended since): sort the new ones, take the larger of
                    // the i-th best old and the i-th worst new, sort that bitonic sequence
                    float nw[kRoom];
#pragma unroll
                    for (int e = 0; e < kRoom; ++e) {
                        const unsigned long long raw = pool[(kept + e) * kTileTok];
                        nw[e] = kept + e < cnt ? __uint_as_float(static_cast<uint32_t>(raw >> 32)) : -INFINITY;
                    }
                    bitonic_sort_desc<kRoom>(nw);
#pragma unroll
                    for (int e = 0; e < N; ++e) best[e] = fmaxf(best[e], nw[N - 1 - e]);
                    bitonic_merge_desc<N>(best);
                    // the K-th best = the smallest of the first K (written so that the list stays in registers:
                    // picking entry K - 1 would index it dynamically)
                    float tau = INFINITY;
#pragma unroll
                    for (int e = 0; e < N; ++e) tau = fminf(tau, e < K ? best[e] : INFINITY);
                    if (tau > -INFINITY) {
                        // exactly K survive: every score above tau, and the earliest of those equal to it
                        int above = 0;
#pragma unroll
                        for (int e = 0; e < N; ++e) above += (e < K && best[e] > tau) ? 1 : 0;
                        int ties = K - above, w = 0;
                        // eight entries per round: their loads go out together (slots past cnt hold old entries or
                        // nothing that matters: their stores land at or behind w and are overwritten or ignored)
#pragma unroll 1
                        for (int e0 = 0; e0 < cnt; e0 += 8) {
                            unsigned long long raw[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) raw[j] = pool[(e0 + j) * kTileTok];
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const float sc = __uint_as_float(static_cast<uint32_t>(raw[j] >> 32));
                                const bool valid = e0 + j < cnt;
                                const bool tie = valid && sc == tau && ties > 0;
                                const bool keep = valid && (sc > tau || tie);
                                ties -= tie ? 1 : 0;
                                if (valid) pool[w * kTileTok] = raw[j];   // w <= e: in place, order preserved
                                w += keep ? 1 : 0;
                            }
                        }
                        cnt = w;
                    }
                    kept = cnt;
                    tau_f = tau;
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.tmem_empty[buf]);
        }
        // (after a timeout the thread still walks through the tile's barriers; every warp leaves together below)
        if (!ok) { set_status(a.status, kDevTimeout); *reinterpret_cast<volatile int*>(&sm.abort) = 1; }

        // the survivors are the selection, already in ascending chunk order; -1 padded
        int ids[N];
#pragma unroll
        for (int e = 0; e < N; ++e) ids[e] = e < cnt ? static_cast<int>(pool[e * kTileTok] & 0xffffffffull) : -1;
        if (tok < s.R) {
            int32_t* sel = a.sel + (static_cast<long long>(pair) * s.R + tok) * K;
#pragma unroll
            for (int e = 0; e < N; ++e)
                if (e < K) sel[e] = ids[e];
        }
        if (a.cnt) {
            // chunk histogram of this tile's entries (selected chunks + the chunks of each token's local window) in the
            // pools' shared memory (every thread holds its ids in registers by now), then one global add per used bin
            int* hist = reinterpret_cast<int*>(lists);
            const bool in_smem = a.nc * sizeof(int) <= sizeof(unsigned long long) * 2 * kMaxK * kTileTok;
            int* gcnt = a.cnt + (static_cast<long long>(ti * kTileTok / a.qb) * pairs + pair) * a.nc;
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (in_smem) {
                for (int x = tid; x < a.nc; x += kTileTok) hist[x] = 0;
                asm volatile("bar.sync 1, 128;" ::: "memory");
            }
            if (tok < s.R) {
                int* dst = in_smem ? hist : gcnt;
#pragma unroll
                for (int e = 0; e < N; ++e)
                    if (ids[e] >= 0) atomicAdd(dst + ids[e], 1);
                const int pos = s.pos0 + tok;
                for (int c = local_lo(pos, s.W, kS) / kS; c <= pos / kS; ++c) atomicAdd(dst + c, 1);
            }
            if (in_smem) {
                asm volatile("bar.sync 1, 128;" ::: "memory");
                for (int x = tid; x < a.nc; x += kTileTok)
                    if (hist[x]) atomicAdd(gcnt + x, hist[x]);
            }
        }
        // the pools' memory (histogram) is free for the next tile; after a timeout every warp leaves here
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (*reinterpret_cast<volatile int*>(&sm.abort)) break;
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 5) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace

bool prefill_select_tc_supports(const Shape& s) {
    return s.K <= kMaxK && static_cast<long long>(s.B) * s.Hq * s.R < (1ll << 31);
}

int launch_prefill_select_tc(const Shape& s, const void* q, const void* landmarks, const float* bias, int32_t* sel,
                             int* status, int* cnt, int qb, int nc, cudaStream_t stream) {
    const int pairs = s.B * s.Hkv;
    CUtensorMap map_q, map_lm;
    if (!make_bf16_2d_map(&map_q, q, static_cast<uint64_t>(s.B) * s.Hq * s.R, kD, 64, kTileTok) ||
        !make_bf16_2d_map(&map_lm, landmarks, static_cast<uint64_t>(s.B) * s.Hl * s.C, kD, 64, kS))
        return HILS_ERR_CUDA;
    const size_t smem = kQBytes + kLmStages * kLmStageBytes + sizeof(unsigned long long) * 2 * kMaxK * kTileTok +
                        sizeof(TcSmem) + 1024;
    static PerDeviceOnce attr_once;
    if (attr_once.pending()) {
        if (cudaFuncSetAttribute(prefill_select_tc_kernel<16, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem)) != cudaSuccess ||
            cudaFuncSetAttribute(prefill_select_tc_kernel<32, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem)) != cudaSuccess ||
            cudaFuncSetAttribute(prefill_select_tc_kernel<16, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem)) != cudaSuccess ||
            cudaFuncSetAttribute(prefill_select_tc_kernel<32, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem)) != cudaSuccess)
            return HILS_ERR_CUDA;
        attr_once.done();
    }
    TcArgs a{s, bias, sel, status, (cnt && qb % kTileTok == 0) ? cnt : nullptr, qb, nc};
    const int tiles = (s.R + kTileTok - 1) / kTileTok;
    const unsigned all_tiles = static_cast<unsigned>(pairs) * tiles;
    const unsigned nsm = static_cast<unsigned>(sm_count());
    const unsigned grid = all_tiles < nsm ? all_tiles : nsm;       // one persistent CTA per SM
    const bool perhead = s.Hl != s.Hkv;
    if (s.K <= 16) {
        if (perhead) prefill_select_tc_kernel<16, true><<<grid, kThreads, smem, stream>>>(map_q, map_lm, a);
        else prefill_select_tc_kernel<16, false><<<grid, kThreads, smem, stream>>>(map_q, map_lm, a);
    } else {
        if (perhead) prefill_select_tc_kernel<32, true><<<grid, kThreads, smem, stream>>>(map_q, map_lm, a);
        else prefill_select_tc_kernel<32, false><<<grid, kThreads, smem, stream>>>(map_q, map_lm, a);
    }
    if (cudaGetLastError() != cudaSuccess) return HILS_ERR_CUDA;
    return a.cnt ? 2 : 1;
}

}  // namespace hils
