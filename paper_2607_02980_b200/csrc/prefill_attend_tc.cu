// Chunk-major gathered attention for prefill on tcgen05 tensor cores (bf16, d = 128, S = 64, G = 4).
//
// A tile is 32 (token, slot) entries of one chunk x 4 heads = 128 query rows (one TMEM lane each).
// Per tile:  S = Q K_c^T (M=128, N=80: 64 keys + the chunk's landmark as key 64, K=128) -> tensor memory;
//            each softmax thread owns one row: mask (local rows are causal), the chunk's own softmax
//            (Eq. HiLS weights, intra-chunk factor), normalised P as bf16 pairs into tensor memory (32 columns behind
//            the slot's scores: shared memory carries neither the write nor the read of P);
//            O = P V_c (M=128, N=128, K=64; A = P from tensor memory, V read from shared memory as an MN-major
//            operand exactly as TMA wrote it) -> tensor memory;
//            bf16 rows and the row's chunk mass (surrogate score, or log Z_swa for the
//            local branch) go to the buffers that prefill_fuse mixes, in entry order: a tile's 128 rows
//            are contiguous there, so every output warp hands its 32 rows to one TMA store per half.
// Warp roles: 0-3 and 4-7 two softmax groups (tiles alternate between them; a warp reads the TMEM lane quarter
// warp % 4), 8-11 output group, 12-15 query gather, 16 K/V loader, 17 MMA issue.
// The gather: a warp's cp.async requests complete at the latency of a loaded L2 and a warp keeps only so many in
// flight, so the rate grows with the number of gathering warps (measured alone: 1 warp 1500 cycles per 32 KB tile, 2
// warps 840, 4 and more 480; inside this kernel about three times that).  TMA boxes of one entry (512 B) cost about
// 86 cycles each and 1-D bulk copies of one row 54: both slower.  More than four gather warps need per-group register
// budgets (setmaxnreg), which measured slower (1.08 ms against 0.73 ms on the 16K-token benchmark shape).
// S/P/O are double buffered, three gathered Q tiles are in flight, K tiles are double and V tiles triple buffered.
#include "internal.h"
#include "tma.cuh"

namespace hils {
namespace {

constexpr int kD = 128;
constexpr int kS = 64;
constexpr int kG = 4;
constexpr int kTok = 32;                        // entries per tile
constexpr int kRows = kTok * kG;                // 128
constexpr int kNS = 80;                         // score columns: 64 keys + landmark (+15 zero rows)
constexpr int kKBytes = kNS * 128 * 2;          // two 64-dim K-blocks of 80 rows
constexpr int kVBytes = kS * kD * 2;            // two boxes of 64 keys x 64 dims
constexpr int kQBytes = kRows * kD * 2;         // 32 KB
constexpr int kPBytes = kRows * 128;            // 16 KB
constexpr int kPCol = 96;                       // probabilities (bf16 pairs, 32 columns) behind the slot's 80 score columns
constexpr int kBatch = 64;                      // tiles whose records and entries are cached in shared memory at a time
                                                // (every batch ends with a drained pipeline: 32 -> 0.701 ms, 48 -> 0.674, 64 -> 0.664
                                                // on the 16K-token benchmark shape; 64 is what fits)
constexpr int kQSlots = 3;                      // gathered Q tiles in flight
constexpr int kVBufs = 3;                       // V tiles in flight (K: 2)
constexpr int kMetaSlots = 16;                  // ring of tile descriptors.  The gather of tile t starts once S(t-3) is done, which
                                                // needs softmax(t-5) under way, hence softmax(t-7) finished, hence P V(t-9) done,
                                                // hence the output of tile t-11 finished: the output group is at most 10 tiles behind
constexpr int kSoftThreads = 256;               // two softmax groups of 128 threads
constexpr int kOutWarp0 = kSoftThreads / 32;    // 8
constexpr int kGatherWarps = 4;
constexpr int kGatherWarp0 = kOutWarp0 + 4;     // 12 .. 15
constexpr int kLoadWarp = kGatherWarp0 + kGatherWarps;   // 16
constexpr int kMmaWarp = kLoadWarp + 1;         // 17, 18: one MMA issuer per tile parity
constexpr int kThreads = (kMmaWarp + 2) * 32;   // 608
constexpr float kLog2e = 1.4426950408889634f;

struct AtcSmem {
    // K tiles live in a ring of 2 (free again after the chunk's last S MMA), V tiles in a ring of kVBufs (free after
    // its last P V MMA, about one epilogue phase later)
    uint64_t k_ready[2];      // K tile landed (TMA bytes) and the landmark row written (one arrival)
    uint64_t v_ready[kVBufs]; // V tile landed
    uint64_t k_empty[2];      // every S MMA that reads this K buffer has completed (relayed by the softmax group)
    uint64_t v_empty[kVBufs]; // every P V MMA that reads this V buffer has completed (relayed by the output group)
    uint64_t q_full[kQSlots]; // gathered Q rows landed (TMA bytes)
    uint64_t q_empty[kQSlots];// the S MMA that reads this Q tile has completed (relayed by the softmax group)
    uint64_t s_full[2];       // S = Q K^T in tensor memory
    uint64_t s_empty[2];      // the slot's softmax group has read S
    uint64_t p_full[2];       // P written to tensor memory
    uint64_t o_full[2];       // O = P V in tensor memory
    uint64_t o_empty[2];      // the output group has read O
    uint32_t tmem_base;
    int abort_flag;
    int tile_meta[kMetaSlots][4];     // pair, chunk, tokens | last tile of its chunk run << 8 | K buffer << 9 | V buffer << 10,
                                      // first entry relative to the query block
    int4 recs[kBatch];
    int ent_s[kBatch * kTok];         // entries of the batch's tiles: (token - block start) << 8 | slot
    int nchunks;                      // distinct (pair, chunk) runs in the current batch
    uint8_t cfirst[kBatch + 4];       // first tile (batch index) of each run; cfirst[nchunks] = tiles in the batch
};

struct AtcArgs {
    Shape s;
    const __nv_bfloat16* q;
    const __nv_bfloat16* lm;
    const float* bias;
    const int* entries;
    const int4* tiles;
    const int* n_tiles;
    float* lam;
    int* status;
    int i0;
    int whole;        // 1: the output buffers cover every query block of the call (rows indexed by global entry)
    int n_run;        // query blocks this launch walks one after the other (> 1 only with whole = 1)
    int qb;           // tokens per query block
};

static_assert(2 * kKBytes + kVBufs * kVBytes + kQSlots * kQBytes + 2 * kPBytes + sizeof(AtcSmem) + 1024 <= 232448,
              "shared memory of the attend kernel");

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__global__ void __launch_bounds__(kThreads, 1)
prefill_attend_tc_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                         const __grid_constant__ CUtensorMap map_o, const AtcArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* kbuf = base;                                   // [2][kKBytes]
    uint8_t* vbuf = kbuf + 2 * kKBytes;                     // [kVBufs][kVBytes]
    uint8_t* qbuf = vbuf + kVBufs * kVBytes;                // [kQSlots][kQBytes]
    uint8_t* obuf = qbuf + kQSlots * kQBytes;               // [2][kPBytes]: staging of the output rows being stored
    AtcSmem& sm = *reinterpret_cast<AtcSmem*>(obuf + 2 * kPBytes);

    const Shape& s = a.s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < kQSlots; ++i) { mbar_init(&sm.q_full[i], kGatherWarps * 32 + kGatherWarps); mbar_init(&sm.q_empty[i], 1); }
        for (int i = 0; i < kVBufs; ++i) { mbar_init(&sm.v_ready[i], 1); mbar_init(&sm.v_empty[i], 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sm.k_ready[i], 2);           // the TMA issuer's arrive.expect_tx + the landmark writer
            mbar_init(&sm.k_empty[i], 2);
            mbar_init(&sm.s_full[i], 1);
            mbar_init(&sm.s_empty[i], 4);
            mbar_init(&sm.p_full[i], 4);
            mbar_init(&sm.o_full[i], 1);
            mbar_init(&sm.o_empty[i], 4);
        }
        mbar_fence_init();
        sm.abort_flag = 0;
        tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v);
        tma_prefetch_desc(&map_o);
    }
    // rows 64..79 of both K-blocks of both K buffers: landmark row + zero rows (TMA never writes them)
    for (int x = tid; x < 2 * 2 * 16 * 8; x += kThreads) {
        const int bufi = x >> 8, kb = (x >> 7) & 1, row = 64 + ((x >> 3) & 15), pc = x & 7;
        *reinterpret_cast<uint4*>(kbuf + bufi * kKBytes + kb * (kNS * 128) + swz128(row, pc)) = make_uint4(0u, 0u, 0u, 0u);
    }
    if (warp == kMmaWarp) tmem_alloc(&sm.tmem_base, 512);
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = sm.tmem_base;

    // Everything above touched only this CTA's own shared and tensor memory, so it may overlap the tail of the
    // previous kernel of the stream (the fusion of the previous query block, which still reads the partial outputs
    // this kernel overwrites, or the inverse-index kernels).  From here on their results are needed.
    pdl_wait();

    // Every role walks the same batches of tiles.  a.n_tiles[blk], a.n_tiles[blk + 1]: first tile of query block blk
    // and of the next one; a launch that walks several blocks takes them in order, so that the CTAs stay on the same
    // block (its gathered Q rows stay in L2).  The walk is instantiated once per role.
    // body(nb, tcount, ccount, t_begin, i0): nb tiles cached in sm.recs, the CTA's running tile and chunk-run counters.
    auto walk = [&](auto&& body) {
        uint32_t tcount = 0, ccount = 0;
        for (int blk = 0; blk < a.n_run; ++blk) {
            const int t_begin = a.n_tiles[blk], n_tiles = a.n_tiles[blk + 1] - t_begin;
            const int i0 = a.i0 + blk * a.qb;
            const long long lo = t_begin + static_cast<long long>(blockIdx.x) * n_tiles / gridDim.x;
            const long long hi = t_begin + static_cast<long long>(blockIdx.x + 1) * n_tiles / gridDim.x;
            for (long long b0 = lo; b0 < hi; b0 += kBatch) {
                const int nb = static_cast<int>(min(static_cast<long long>(kBatch), hi - b0));
                for (int x = tid; x < nb; x += kThreads) sm.recs[x] = a.tiles[b0 + x];
                // A list starts on a tile boundary of the global entry space, so the entries of tile t are
                // entries[32 t .. 32 t + 31]: the batch's entries are one contiguous run, fetched now, all at once (a
                // load per tile inside the gather loop waited several thousand cycles under the partial-output stores).
                for (int x = tid; x < nb * kTok; x += kThreads) sm.ent_s[x] = a.entries[b0 * kTok + x];
                __syncthreads();
                if (sm.abort_flag) return;
                if (warp == 0) {
                    // table of chunk runs: where each run of tiles of one (pair, chunk) starts
                    int basec = 0;
                    for (int w = 0; w < (kBatch + 31) / 32; ++w) {
                        const int x = w * 32 + lane;
                        const bool nw = x < nb && (x == 0 || sm.recs[x].x != sm.recs[x - 1].x || sm.recs[x].y != sm.recs[x - 1].y);
                        const unsigned m = __ballot_sync(kFullMask, nw);
                        if (nw) sm.cfirst[basec + __popc(m & ((1u << lane) - 1u))] = static_cast<uint8_t>(x);
                        basec += __popc(m);
                    }
                    if (lane == 0) { sm.cfirst[basec] = static_cast<uint8_t>(nb); sm.nchunks = basec; }
                }
                __syncthreads();
                body(nb, tcount, ccount, t_begin, i0);
                // every role advances the shared counters identically
                tcount += static_cast<uint32_t>(nb);
                ccount += static_cast<uint32_t>(sm.nchunks);
                __syncthreads();
                if (sm.abort_flag) return;
            }
        }
    };

    auto gather_role = [&]() {
        // ================================================================ Q gather (four warps)
        // The tile's 128 rows (entry-major, head-minor) are 64 cp.async instructions of two 256-byte rows (a half-warp
        // each, both of one entry); warp gw issues numbers 16 gw .. 16 gw + 15.  Lane l < 8 holds entry 8 gw + l and
        // hands its token to the warp by a uniform shuffle: no address table, no barrier between the gather warps.
        const int gw = warp - kGatherWarp0;
        constexpr int kPerWarp = 64 / kGatherWarps;
        const int j0 = gw * kPerWarp, j1 = j0 + kPerWarp;
        const int e0 = j0 >> 1;                                      // first entry this warp touches
        const int el = min(e0 + (lane & 7), kTok - 1);
        const int p16 = lane & 15, hh = lane >> 4;
        const long long hstride = static_cast<long long>(s.R) * kD;
        walk([&](int nb, uint32_t tcount, uint32_t ccount, int t_begin, int i0) {
            uint32_t tc = tcount;
            bool dead = false;
            int ck = 0;                        // chunk run (ordinal within the batch) of the current tile
            for (int ti = 0; ti < nb; ++ti) {
                const int4 rec = sm.recs[ti];
                const int pair = rec.x, ntok = rec.w;
                // this lane's entry (rows past a ragged tile's last entry repeat that entry)
                const int e = sm.ent_s[ti * kTok + min(el, ntok - 1)];
                const uint32_t qs = tc % kQSlots, ms = tc % kMetaSlots;
                if (tc >= kQSlots && !mbar_wait(&sm.q_empty[qs], ((tc / kQSlots) - 1) & 1)) { dead = true; break; }
                if (*reinterpret_cast<volatile int*>(&sm.abort_flag)) { dead = true; break; }
                if (gw == 0 && lane == 0) {
                    // A tcgen05.commit costs the issuing thread about a hundred cycles, so only the two the epilogue
                    // groups wait on are issued; those groups pass "this Q slot / K buffer / V buffer is free" on.
                    if (ti >= sm.cfirst[ck + 1]) ++ck;
                    const bool last = ti + 1 >= sm.cfirst[ck + 1];
                    // The K buffer of a chunk run is free when the score MMAs of the run's last tile of EITHER parity are
                    // done (the two parities have an issuing thread each, and a thread's MMAs complete in order): those
                    // two tiles arrive once each on k_empty, a run of a single tile twice.
                    const int karr = (ti + 2 >= sm.cfirst[ck + 1] ? 1 : 0) + (sm.cfirst[ck + 1] - sm.cfirst[ck] == 1 ? 1 : 0);
                    const uint32_t cc = ccount + static_cast<uint32_t>(ck);
                    sm.tile_meta[ms][0] = pair; sm.tile_meta[ms][1] = rec.y;
                    sm.tile_meta[ms][2] = ntok | (last ? 256 : 0) | static_cast<int>((cc & 1u) << 9) | static_cast<int>((cc % kVBufs) << 10) | (karr << 12);
                    sm.tile_meta[ms][3] = rec.z - (a.whole ? 0 : t_begin * kTok);
                }
                {
                    const uint32_t qaddr = smem_u32(qbuf + qs * kQBytes) + (p16 >> 3) * 16384;
                    const __nv_bfloat16* qb0 = a.q + (static_cast<long long>(pair / s.Hkv) * s.Hq + (pair % s.Hkv) * kG + hh) * hstride +
                                               static_cast<long long>(i0) * kD + p16 * 8;
                    // the tokens of the warp's entries first (shuffles and copies are both ordered operations: interleaved
                    // they would run strictly one after the other)
                    int tokv[kPerWarp / 2];
#pragma unroll
                    for (int k = 0; k < kPerWarp / 2; ++k) tokv[k] = __shfl_sync(kFullMask, e, k) >> 8;
#pragma unroll
                    for (int jj = 0; jj < kPerWarp; ++jj) {
                        const int j = j0 + jj;
                        const int row = 2 * j + hh;
                        const __nv_bfloat16* src = qb0 + (2 * j & 3) * hstride + static_cast<long long>(tokv[jj >> 1]) * kD;
                        cp_async16(qaddr + swz128(row, p16 & 7), src);
                    }
                }
                // The tile's barrier hears from every gather thread when that thread's copies have landed (no thread
                // waits for them), and from one lane per warp for the tile's descriptor written above.
                asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(&sm.q_full[qs])) : "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.q_full[qs]);
                ++tc;
            }
            if (dead && lane == 0) { set_status(a.status, kDevTimeout); atomicExch(&sm.abort_flag, 1); }
        });
    };

    // (called at the end of every role)
    auto finish = [&]() {
        tc_fence_before_sync();
        __syncthreads();
        tc_fence_after_sync();
        if (warp == kMmaWarp) tmem_dealloc(tmem_base, 512);
    };

    if (warp < kOutWarp0) {
        // ================================================================ softmax: one row per thread
        // Group g (warps 4g .. 4g+3) turns the scores of the tiles in S/P/O slot g into probabilities: the two
        // groups work on consecutive tiles at the same time.
        const uint32_t grp = static_cast<uint32_t>(warp >> 2);
        const int row = (warp & 3) * 32 + lane;
        const uint32_t t_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16) + grp * 128;
        const int tk = row >> 2, hd = row & 3;
        const float sl2 = s.scale * kLog2e;
        const int lh = (s.Hl == s.Hkv) ? 0 : hd;
        walk([&](int nb, uint32_t tcount, uint32_t, int, int i0) {
            bool ok = true;
            for (int ti = static_cast<int>((grp ^ tcount) & 1u); ti < nb && ok; ti += 2) {
                const uint32_t tcv = tcount + ti;                      // (tcv & 1) == grp
                ok = mbar_wait(&sm.s_full[grp], (tcv >> 1) & 1);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t ms = tcv % kMetaSlots;
                const int pair = sm.tile_meta[ms][0], c = sm.tile_meta[ms][1];
                // the tile's score MMAs are done: its gathered rows, and its chunk's K tile after the chunk's last tile,
                // may be overwritten
                if ((warp & 3) == 0 && lane == 0) {
                    const int flags = sm.tile_meta[ms][2];
                    mbar_arrive(&sm.q_empty[tcv % kQSlots]);
                    for (int x = (flags >> 12) & 3; x > 0; --x) mbar_arrive(&sm.k_empty[(flags >> 9) & 1]);
                }
                const int orow0 = sm.tile_meta[ms][3] * kG;          // first row of the tile in the output buffers
                const int e = sm.ent_s[ti * kTok + min(tk, (sm.tile_meta[ms][2] & 255) - 1)];
                const int il = e >> 8, slot = e & 255;
                const bool local = slot >= s.K;                            // a chunk of the local window: mass = its exact log-sum-exp
                const int lim = local ? s.pos0 + i0 + il - c * kS : kS - 1;   // last visible key of the chunk
                // the 64 key scores and the surrogate score columns: the landmark of this row's head (key 64 + hd)
                // or the shared one (key 64); warp-uniform addresses, the lane picks its column
                float v[64];
                float lm4[4];
                tmem_ld64_4(t_lane, t_lane + 64, v, lm4);
                const float lmk = lh == 0 ? lm4[0] : (lh == 1 ? lm4[1] : (lh == 2 ? lm4[2] : lm4[3]));
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.s_empty[grp]);
                if (__any_sync(kFullMask, local)) {
#pragma unroll
                    for (int j = 0; j < 64; ++j)
                        if (j > lim) v[j] = -INFINITY;
                }
                // four independent chains of three-input maxima
                float mx[4] = {v[0], v[1], v[2], v[3]};
#pragma unroll
                for (int j = 4; j < 60; j += 8) {
                    mx[0] = fmax3(mx[0], v[j], v[j + 1]);
                    mx[1] = fmax3(mx[1], v[j + 2], v[j + 3]);
                    mx[2] = fmax3(mx[2], v[j + 4], v[j + 5]);
                    mx[3] = fmax3(mx[3], v[j + 6], v[j + 7]);
                }
                mx[0] = fmax3(mx[0], v[60], v[61]);
                mx[1] = fmax3(mx[1], v[62], v[63]);
                const float m = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                const float2 sl22 = make_float2(sl2, sl2);
                const float2 nms2 = make_float2(-m * sl2, -m * sl2);
                // exponentials in place, two lanes of arithmetic per instruction; four chains for the row sum
                float2 zp[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float2 x = __ffma2_rn(make_float2(v[2 * j], v[2 * j + 1]), sl22, nms2);
                    v[2 * j] = ex2_approx(x.x);
                    v[2 * j + 1] = ex2_approx(x.y);
                    zp[j & 3] = __fadd2_rn(zp[j & 3], make_float2(v[2 * j], v[2 * j + 1]));
                }
                const float2 z2 = __fadd2_rn(__fadd2_rn(zp[0], zp[1]), __fadd2_rn(zp[2], zp[3]));
                const float z = z2.x + z2.y;
                const float zi = 1.f / z;
                const float2 zi2 = make_float2(zi, zi);
                // the P V product of this slot's previous tile must have read its probabilities
                if (tcv >= 2) {
                    ok = mbar_wait(&sm.o_full[grp], ((tcv >> 1) - 1) & 1);
                    if (!ok) break;
                }
#pragma unroll
                for (int pc = 0; pc < 4; ++pc) {
                    uint32_t pk[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float2 p = __fmul2_rn(make_float2(v[pc * 16 + 2 * j], v[pc * 16 + 2 * j + 1]), zi2);
                        pk[j] = pack_bf16(p.x, p.y);
                    }
                    tmem_st8(t_lane + kPCol + pc * 8, pk);
                }
                // chunk mass of the row (rows of a ragged tile's padding land in the list's padding)
                const float bb = (a.bias && c < s.C)
                    ? a.bias[(static_cast<long long>(pair / s.Hkv) * s.Hl + (pair % s.Hkv) * (s.Hl / s.Hkv) + lh) * s.C + c] : 0.f;
                a.lam[orow0 + row] = local ? m * s.scale + __logf(z) : lmk * s.scale + bb;
                tmem_wait_st();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.p_full[grp]);
            }
            if (!ok && lane == 0) { set_status(a.status, kDevTimeout); atomicExch(&sm.abort_flag, 1); }
        });
        finish();
    } else if (warp < kGatherWarp0) {
        // ================================================================ output group: O = P V -> bf16 rows
        // The warp's 32 rows of the staging buffer (4 KB, swizzled as the output map expects) take 64 columns at a
        // time; one TMA store per half writes 32 full rows.
        const int ow = warp - kOutWarp0;
        const int row = ow * 32 + lane;
        const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(ow * 32) << 16);
        const uint64_t pol = l2_policy_evict_first();
        uint8_t* wstg = obuf + ow * 4096;            // columns 0..63; + kPBytes: columns 64..127
        walk([&](int nb, uint32_t tcount, uint32_t, int, int) {
            bool ok = true;
            for (int ti = 0; ti < nb && ok; ++ti) {
                const uint32_t tcv = tcount + ti, sl = tcv & 1u;
                ok = mbar_wait(&sm.o_full[sl], (tcv >> 1) & 1);
                if (!ok) break;
                tc_fence_after_sync();
                const int orow0 = sm.tile_meta[tcv % kMetaSlots][3] * kG;
                if (ow == 0 && lane == 0) {
                    // the tile's P V MMAs are done: after the chunk's last tile its V tile may be overwritten
                    const int flags = sm.tile_meta[tcv % kMetaSlots][2];
                    if (flags & 256) mbar_arrive(&sm.v_empty[(flags >> 10) & 3]);
                }
                // The accumulator leaves tensor memory in four quarters of 32 columns; the load of the next quarter runs
                // under the packing and staging of the current one.
                uint32_t va[32], vb[32];
                const uint32_t o_col = t_lane + 256 + sl * 128;
                tmem_ld32_issue(o_col, va);
                tmem_ld_wait32(va);
                tmem_ld32_issue(o_col + 32, vb);
                // the previous tile's stores (lane 0: columns 0..63, lane 1: 64..127) must have read the staging rows
                if (lane < 2) bulk_wait_read<0>();
                __syncwarp();
                auto stage = [&](const uint32_t (&v)[32], int q) {
                    // quarter q: columns 32 q .. 32 q + 31 -> four 16-byte pieces of the row's half q / 2
#pragma unroll
                    for (int pc = 0; pc < 4; ++pc) {
                        uint4 w;
                        w.x = pack_bf16(__uint_as_float(v[8 * pc]), __uint_as_float(v[8 * pc + 1]));
                        w.y = pack_bf16(__uint_as_float(v[8 * pc + 2]), __uint_as_float(v[8 * pc + 3]));
                        w.z = pack_bf16(__uint_as_float(v[8 * pc + 4]), __uint_as_float(v[8 * pc + 5]));
                        w.w = pack_bf16(__uint_as_float(v[8 * pc + 6]), __uint_as_float(v[8 * pc + 7]));
                        *reinterpret_cast<uint4*>(obuf + (q >> 1) * kPBytes + swz128(row, (q & 1) * 4 + pc)) = w;
                    }
                };
                stage(va, 0);
                tmem_ld_wait32(vb);
                tmem_ld32_issue(o_col + 64, va);
                stage(vb, 1);
                tmem_ld_wait32(va);
                tmem_ld32_issue(o_col + 96, vb);
                stage(va, 2);
                tmem_ld_wait32(vb);
                // the accumulator is free for the slot's next tile
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.o_empty[sl]);
                stage(vb, 3);
                fence_proxy_async_smem();
                __syncwarp();
                if (lane < 2) {
                    tma_store_2d(&map_o, wstg + lane * kPBytes, lane * 64, orow0 + ow * 32, pol);
                    bulk_commit();
                }
            }
            if (!ok && lane == 0) { set_status(a.status, kDevTimeout); atomicExch(&sm.abort_flag, 1); }
        });
        finish();
    } else if (warp < kLoadWarp) {
        gather_role();
        finish();
    } else {
        if (warp == kLoadWarp) {
            // ================================================================ K/V loader (one warp)
            // One chunk run after the other: wait until the run's K and V buffers are free, request the tiles (they
            // complete on k_ready / v_ready, which only the MMA warp waits for), write the landmark row(s).
            const int per = s.Hl / s.Hkv;      // landmark rows per chunk: 1, or one per query head (App. C)
            auto lm_piece = [&](int pr, int ch, int x) {
                // 16-byte piece x % 16 of landmark head x / 16 of KV-head pair pr, chunk ch
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (ch < s.C) {
                    const long long lrow = (static_cast<long long>(pr / s.Hkv) * s.Hl + (pr % s.Hkv) * per + (x >> 4)) * s.C + ch;
                    v = *reinterpret_cast<const uint4*>(a.lm + lrow * kD + (x & 15) * 8);
                }
                return v;
            };
            walk([&](int, uint32_t, uint32_t ccount, int, int) {
                const int nch = sm.nchunks;
                bool dead = false;
                // landmark pieces of the current run (piece x = lane + 32 r of the `per` rows, 16 pieces each),
                // fetched a run ahead
                uint4 lm_cur[2] = {make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u)};
                if (nch > 0) {
                    const int4 r0 = sm.recs[0];
#pragma unroll
                    for (int r = 0; r < 2; ++r)
                        if (lane + 32 * r < per * 16) lm_cur[r] = lm_piece(r0.x, r0.y, lane + 32 * r);
                }
                for (int ck = 0; ck < nch; ++ck) {
                    const uint32_t cc = ccount + static_cast<uint32_t>(ck);
                    const int4 rec = sm.recs[sm.cfirst[ck]];
                    const int pair = rec.x, c = rec.y;
                    const uint32_t cbuf = cc & 1u, vb = cc % kVBufs;
                    if (lane == 0) {
                        if (cc >= 2 && !mbar_wait(&sm.k_empty[cbuf], ((cc >> 1) - 1) & 1)) dead = true;
                        if (!dead && cc >= kVBufs && !mbar_wait(&sm.v_empty[vb], ((cc / kVBufs) - 1) & 1)) dead = true;
                        if (!dead) {
                            const int row = pair * s.T + c * kS;
                            mbar_expect_tx(&sm.k_ready[cbuf], 2 * 8192);
                            tma_load_2d(kbuf + cbuf * kKBytes, &map_k, &sm.k_ready[cbuf], 0, row);
                            tma_load_2d(kbuf + cbuf * kKBytes + kNS * 128, &map_k, &sm.k_ready[cbuf], 64, row);
                            mbar_expect_tx(&sm.v_ready[vb], kVBytes);
                            tma_load_2d(vbuf + vb * kVBytes, &map_v, &sm.v_ready[vb], 0, row);
                            tma_load_2d(vbuf + vb * kVBytes + 8192, &map_v, &sm.v_ready[vb], 64, row);
                            // warm L2 with the K/V rows of the run after the next one
                            if (ck + 2 < nch) {
                                const int4 r2 = sm.recs[sm.cfirst[ck + 2]];
                                const int row2 = r2.x * s.T + r2.y * kS;
                                tma_prefetch_l2_2d(&map_k, 0, row2);
                                tma_prefetch_l2_2d(&map_k, 64, row2);
                                tma_prefetch_l2_2d(&map_v, 0, row2);
                                tma_prefetch_l2_2d(&map_v, 64, row2);
                            }
                        }
                    }
                    dead = __shfl_sync(kFullMask, dead ? 1 : 0, 0) != 0;
                    if (dead || *reinterpret_cast<volatile int*>(&sm.abort_flag)) { dead = true; break; }
                    // landmark row(s) (keys 64 .. 64 + per - 1) of both K-blocks: the buffer is free (its previous
                    // user's MMAs are done) and TMA never writes these rows.  V stays as TMA writes it (keys x dims):
                    // the second MMA reads it as an MN-major operand; keys past the end of the sequence hold other
                    // rows' data (or TMA zero fill) and meet probabilities of 0.
                    const bool have_next = ck + 1 < nch;
                    const int4 r1 = have_next ? sm.recs[sm.cfirst[ck + 1]] : make_int4(0, 0, 0, 0);
#pragma unroll
                    for (int r = 0; r < 2; ++r) {
                        const int x = lane + 32 * r;
                        if (x < per * 16) {
                            const int pc = x & 15;
                            *reinterpret_cast<uint4*>(kbuf + cbuf * kKBytes + (pc >> 3) * (kNS * 128) + swz128(64 + (x >> 4), pc & 7)) = lm_cur[r];
                            if (have_next) lm_cur[r] = lm_piece(r1.x, r1.y, x);
                        }
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm.k_ready[cbuf]);
                }
                if (dead && lane == 0) { set_status(a.status, kDevTimeout); atomicExch(&sm.abort_flag, 1); }
            });
        } else {
            // ================================================================ MMA issuers (one thread per tile parity)
            // The issuing thread is the critical path of a tile (it is blocked while the tensor pipe takes its MMAs and
            // every barrier test is a shared-memory round trip), so the tiles are split between two of them: warp 17
            // serves the tiles in S/P/O slot 0, warp 18 those in slot 1.  Each commits its own s_full / o_full; a
            // thread's MMAs complete in order, which is what the K-buffer hand-back above relies on.
            const uint32_t par = static_cast<uint32_t>(warp - kMmaWarp);
            walk([&](int nb, uint32_t tcount, uint32_t ccount, int, int) {
                if (lane != 0) return;
                constexpr uint32_t idesc_s = umma_idesc_bf16(kRows, kNS);
                constexpr uint32_t idesc_o = umma_idesc_bf16(kRows, kD) | kUmmaBMnMajor;
                const uint32_t sl = par;
                bool ok = true;
                // Two in-order queues (S MMAs, O MMAs) over this thread's tiles, served by polling: an O MMA whose
                // probabilities are ready is never held up by a Q tile that has not arrived yet, and vice versa.  The
                // chunk run of a tile (its K / V buffers) is looked up in the batch's run table.
                int ns = static_cast<int>((par ^ tcount) & 1u), no = ns;       // next tile (batch index) for S / O
                int ck_s = 0, ck_o = 0, run_s = -1, run_o = -1;                 // run of that tile; last run waited for
                uint32_t idle = 0;
                while (no < nb && ok) {
                    bool progressed = false;
                    if (ns < nb) {
                        const uint32_t tcv = tcount + ns, qs = tcv % kQSlots;
                        while (ns >= sm.cfirst[ck_s + 1]) ++ck_s;
                        const uint32_t cc = ccount + static_cast<uint32_t>(ck_s);
                        bool ready = mbar_test_wait(&sm.q_full[qs], (tcv / kQSlots) & 1);
                        if (ready && run_s != ck_s) ready = mbar_test_wait(&sm.k_ready[cc & 1u], (cc >> 1) & 1);
                        if (ready && tcv >= 2) ready = mbar_test_wait(&sm.s_empty[sl], ((tcv >> 1) - 1) & 1);
                        if (ready) {
                            run_s = ck_s;
                            // the gathered rows were written by cp.async (generic proxy), the MMA reads them through
                            // the async proxy
                            fence_proxy_async_smem();
                            tc_fence_after_sync();
                            const uint32_t qa = smem_u32(qbuf + qs * kQBytes), ka = smem_u32(kbuf + (cc & 1u) * kKBytes);
#pragma unroll
                            for (int ks = 0; ks < 8; ++ks)
                                umma_bf16(tmem_base + sl * 128, umma_desc_k128(qa + (ks >> 2) * 16384 + (ks & 3) * 32),
                                          umma_desc_k128(ka + (ks >> 2) * (kNS * 128) + (ks & 3) * 32), idesc_s, ks > 0 ? 1u : 0u);
                            umma_commit(&sm.s_full[sl]);
                            ns += 2;
                            progressed = true;
                        }
                    }
                    if (no < ns) {
                        const uint32_t tcv = tcount + no;
                        while (no >= sm.cfirst[ck_o + 1]) ++ck_o;
                        const uint32_t cco = ccount + static_cast<uint32_t>(ck_o);
                        bool ready = mbar_test_wait(&sm.p_full[sl], (tcv >> 1) & 1);
                        if (ready && run_o != ck_o) ready = mbar_test_wait(&sm.v_ready[cco % kVBufs], (cco / kVBufs) & 1);
                        if (ready && tcv >= 2) ready = mbar_test_wait(&sm.o_empty[sl], ((tcv >> 1) - 1) & 1);
                        if (ready) {
                            run_o = ck_o;
                            tc_fence_after_sync();
                            const uint32_t va = smem_u32(vbuf + (cco % kVBufs) * kVBytes);
                            // P from tensor memory (columns kPCol.. of the slot: 8 columns = 16 keys per step), V from
                            // shared memory, 16 keys per step = two 8-row groups
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks)
                                umma_bf16_ts(tmem_base + 256 + sl * 128, tmem_base + sl * 128 + kPCol + ks * 8,
                                             umma_desc_mn128(va + ks * 2048, 8192u, 1024u), idesc_o, ks > 0 ? 1u : 0u);
                            umma_commit(&sm.o_full[sl]);
                            no += 2;
                            progressed = true;
                        }
                    }
                    if (progressed) {
                        idle = 0;
                    } else {
                        if (++idle > kSpinLimit) ok = false;          // bounded: give up instead of hanging
                        if (idle > 64) __nanosleep(idle > 4096 ? 256 : 32);
                    }
                }
                if (!ok) { set_status(a.status, kDevTimeout); atomicExch(&sm.abort_flag, 1); }
            });
        }
        finish();
    }
}

}  // namespace

int attend_tc_tile_tokens() { return kTok; }

int launch_prefill_attend_tc(const Shape& s, const void* q, const void* maps, const void* landmarks,
                             const float* bias, const int* entries, const void* tiles, const int* n_tiles, float* lam,
                             int* status, int i0, int whole, int n_run, int qb, cudaStream_t stream) {
    const CUtensorMap* m = static_cast<const CUtensorMap*>(maps);
    const size_t smem = 2 * kKBytes + kVBufs * kVBytes + kQSlots * kQBytes + 2 * kPBytes + sizeof(AtcSmem) + 1024;
    static PerDeviceOnce attr_once;
    if (attr_once.pending()) {
        if (cudaFuncSetAttribute(prefill_attend_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem)) != cudaSuccess)
            return HILS_ERR_CUDA;
        attr_once.done();
    }
    AtcArgs a{s, static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(landmarks), bias, entries,
              static_cast<const int4*>(tiles), n_tiles, lam, status, i0, whole, n_run, qb};
    if (launch_pdl(prefill_attend_tc_kernel, dim3(sm_count()), dim3(kThreads), smem, stream, m[0], m[1], m[2], a) != cudaSuccess)
        return HILS_ERR_CUDA;
    if (cudaGetLastError() != cudaSuccess) return HILS_ERR_CUDA;
    return 1;
}

}  // namespace hils
