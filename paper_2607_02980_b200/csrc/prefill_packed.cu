// Query-major prefill with adjacent-query packing (Sec. 4.2 "Hardware-Efficient Kernel Design"; App. "Chunk Overlap").
//
// A tile is M = 16 adjacent tokens x the G = 4 query heads of one KV head: 64 rows, one 16-row MMA tile per warp.  The
// tile walks the UNION of the chunks its tokens selected (plus the chunks of their local windows); for every chunk all
// 64 rows are scored against its 64 keys, a row that did not select the chunk gets weight zero (pair masking), and the
// retrieval-weighted mix of Eq. HiLS weights is kept in registers across the chunks: per row a running maximum of the
// mixing logits (the per-head surrogate score of a selected chunk, the exact log mass of a local one), the running
// sum of their exponentials and the 128 accumulated output values, rescaled when the maximum moves.  `out` and `lse`
// are written once; no partial outputs, no inverse index, no second kernel.
//
// What it costs: every chunk of the union is attended by all 16 tokens, so the MMA work is |union| / K times the
// chunk-major kernel's.  On queries that share most of their chunks (the regime the paper measures, 80-93 % overlap)
// that factor is small; on independent queries the union approaches 16 K chunks and the chunk-major path is the one
// to use.  This path is chosen explicitly (HILS_IMPL_PACKED); results agree with the chunk-major kernels up to the
// order of the fp32 sums.
//
// Roles: 4 compute warps (mma.sync m16n8k16, bf16 x bf16 -> fp32; the per-chunk tiles are 16 x 64 x 128 and 16 x 128 x 64,
// too small a share of a 128-row tcgen05 tile each to be worth tensor memory round trips), 1 producer warp that
// streams the chunks' K and V tiles (TMA) and landmark rows (bulk copies) through a 3-stage ring.  Two CTAs per SM.
#include "internal.h"
#include "tma.cuh"

namespace hils {
namespace {

constexpr int kD = 128;
constexpr int kS = 64;
constexpr int kG = 4;
constexpr int kM = 16;                         // adjacent tokens per tile
constexpr int kWarps = kM * kG / 16;           // compute warps: 16 rows each
constexpr int kThreads = (kWarps + 1) * 32;
constexpr int kStages = 3;
constexpr int kLmBytes = 256;                  // one landmark row per chunk
constexpr int kStageBytes = 2 * kS * kD * 2 + kLmBytes;
constexpr int kMaxC = 4096;                    // chunks a pair may have (token masks live in shared memory)
constexpr int kMaxUnion = kM * 64;             // K <= 64
constexpr int kMaxLocal = 16;
constexpr float kLog2e = 1.4426950408889634f;

struct PkArgs {
    Shape s;
    const __nv_bfloat16* q;
    const __nv_bfloat16* lm;
    const float* bias;
    const int32_t* sel;
    __nv_bfloat16* out;
    float* lse;
    int* status;
};

struct PkSmem {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint32_t tokmask[kMaxC / 2];               // 16 token bits per chunk, two chunks per word
    uint16_t ulist[kMaxUnion];                 // union of the tile's selected chunks, ascending
    int n_union;
    int dead;
};

// S = Q K^T, 16 rows x 64 keys; the K tile is two 128B-swizzled boxes of 64 dims, 8192 bytes apart.
// sc[nt][0..1]: row lane / 4, keys 8 nt + 2 (lane % 4) + {0, 1}; sc[nt][2..3]: row lane / 4 + 8.
__device__ __forceinline__ void qk_tile16(const uint32_t (&aq)[8][4], uint32_t ks_addr, int lane, float (&sc)[8][4]) {
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
        sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
        for (int kp = 0; kp < 4; ++kp) {
            const int row = nt * 8 + (lane & 7);
            const int dim = kp * 32 + (lane >> 3) * 8;
            const uint32_t addr = ks_addr + (dim >> 6) * 8192 + swz128(row, (dim & 63) >> 3);
            uint32_t r0, r1, r2, r3;
            ldmatrix_x4(addr, r0, r1, r2, r3);
            mma_bf16_16816(sc[nt], aq[2 * kp], r0, r1);
            mma_bf16_16816(sc[nt], aq[2 * kp + 1], r2, r3);
        }
    }
}

// O += P V, 16 rows x 128 dims over 64 keys; p as qk_tile16 leaves it (already weighted).
__device__ __forceinline__ void pv_tile16(const float (&p)[8][4], uint32_t vs_addr, int lane, float (&o)[16][4]) {
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
        const uint32_t ap[4] = {pack_bf16(p[2 * kk][0], p[2 * kk][1]), pack_bf16(p[2 * kk][2], p[2 * kk][3]),
                                pack_bf16(p[2 * kk + 1][0], p[2 * kk + 1][1]), pack_bf16(p[2 * kk + 1][2], p[2 * kk + 1][3])};
#pragma unroll
        for (int dp = 0; dp < 8; ++dp) {
            const int mat = lane >> 3;
            const int row = kk * 16 + (mat & 1) * 8 + (lane & 7);
            const int dim = dp * 16 + (mat >> 1) * 8;
            const uint32_t addr = vs_addr + (dim >> 6) * 8192 + swz128(row, (dim & 63) >> 3);
            uint32_t r0, r1, r2, r3;
            ldmatrix_x4_trans(addr, r0, r1, r2, r3);
            mma_bf16_16816(o[2 * dp], ap, r0, r1);
            mma_bf16_16816(o[2 * dp + 1], ap, r2, r3);
        }
    }
}

__device__ __forceinline__ void bulk_load(void* sdst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(sdst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

__global__ void __launch_bounds__(kThreads, 2)
prefill_packed_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                      const PkArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    PkSmem& sm = *reinterpret_cast<PkSmem*>(ring + kStages * (kStageBytes + 768));   // stages 1024-byte aligned
    constexpr int kStride = kStageBytes + 768;
    const Shape& s = a.s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int pairs = s.B * s.Hkv;
    const int tiles_per_seq = (s.R + kM - 1) / kM;
    const int n_tiles = pairs * tiles_per_seq;
    const int K = s.K;
    const int NL = (s.W - 1 + kS - 1) / kS + 1;         // chunks a local window can touch

    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], kWarps); }
        mbar_fence_init();
        sm.dead = 0;
        tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v);
    }
    __syncthreads();

    uint32_t n_item = 0;                     // items so far, over all tiles of this CTA (ring phase)
    for (int idx = blockIdx.x; idx < n_tiles; idx += gridDim.x) {
        // heavy tiles (late tokens: long candidate lists, large unions) first
        const int tt = tiles_per_seq - 1 - idx / pairs, pair = idx % pairs;
        const int b = pair / s.Hkv, g = pair % s.Hkv;
        const int tok0 = tt * kM;
        const int pos_first = s.pos0 + tok0, pos_last = s.pos0 + min(s.R, tok0 + kM) - 1;
        const int ci = pos_first / kS;                              // the tile's own chunk (kM divides kS)
        const int lc_min = local_lo(pos_first, s.W, kS) / kS;       // first chunk of any token's local window
        const int ncand_max = local_lo(pos_last, s.W, kS) / kS;     // candidates of the tile's last token
        const int n_local = ci - lc_min + 1;

        // ---- the union of the selections: token masks per chunk, then the ascending list
        for (int x = tid; x < (ncand_max + 1) / 2 + 1 && x < kMaxC / 2; x += kThreads) sm.tokmask[x] = 0u;
        __syncthreads();
        for (int x = tid; x < kM * K; x += kThreads) {
            const int t = x / K, k = x % K;
            if (tok0 + t < s.R) {
                const int c = a.sel[(static_cast<long long>(pair) * s.R + tok0 + t) * K + k];
                if (c >= 0 && c < ncand_max) atomicOr(&sm.tokmask[c >> 1], 1u << ((c & 1) * 16 + t));
            }
        }
        __syncthreads();
        if (warp == kWarps) {
            int n = 0;
            for (int c0 = 0; c0 < ncand_max; c0 += 32) {
                const int c = c0 + lane;
                const bool used = c < ncand_max && ((sm.tokmask[c >> 1] >> ((c & 1) * 16)) & 0xffffu) != 0u;
                const unsigned bal = __ballot_sync(kFullMask, used);
                if (used) sm.ulist[n + __popc(bal & ((1u << lane) - 1u))] = static_cast<uint16_t>(c);
                n += __popc(bal);
            }
            if (lane == 0) sm.n_union = n;
        }
        __syncthreads();
        const int n_union = sm.n_union;
        const int n_items = n_local + n_union;
        // item j: j < n_local: local chunk lc_min + j; else union chunk ulist[j - n_local]
        auto item_chunk = [&](int j) { return j < n_local ? lc_min + j : static_cast<int>(sm.ulist[j - n_local]); };

        if (warp == kWarps) {
            // ------------------------------------------------------------------ producer (one lane)
            if (lane == 0) {
                bool ok = true;
                for (int j = 0; j < n_items && ok; ++j) {
                    const uint32_t it = n_item + j, st = it % kStages;
                    if (it >= kStages) ok = mbar_wait(&sm.empty[st], ((it / kStages) - 1) & 1);
                    if (!ok) break;
                    const int c = item_chunk(j);
                    const int row = pair * s.T + c * kS;
                    uint8_t* dst = ring + st * kStride;
                    const bool selected = j >= n_local;
                    mbar_expect_tx(&sm.full[st], 2 * kS * kD * 2 + (selected ? kLmBytes : 0));
                    tma_load_2d(dst, &map_k, &sm.full[st], 0, row);
                    tma_load_2d(dst + 8192, &map_k, &sm.full[st], 64, row);
                    tma_load_2d(dst + 16384, &map_v, &sm.full[st], 0, row);
                    tma_load_2d(dst + 24576, &map_v, &sm.full[st], 64, row);
                    if (selected)
                        bulk_load(dst + 32768, a.lm + (static_cast<long long>(pair) * s.C + c) * kD, kLmBytes, &sm.full[st]);
                }
                if (!ok) { set_status(a.status, kDevTimeout); atomicExch(&sm.dead, 1); }
            }
        } else {
            // ------------------------------------------------------------------ compute: 16 rows per warp
            const int gq = lane >> 2, t = lane & 3;
            // rows gq and gq + 8 of the warp: token warp * 4 + row / 4, head row % 4
            const int tl0 = warp * 4 + (gq >> 2), tl1 = tl0 + 2, hd = gq & 3;
            const int tokA = tok0 + tl0, tokB = tok0 + tl1;
            const bool liveA = tokA < s.R, liveB = tokB < s.R;
            const int posA = s.pos0 + tokA, posB = s.pos0 + tokB;
            const int lcA = local_lo(posA, s.W, kS) / kS, lcB = local_lo(posB, s.W, kS) / kS;
            uint32_t aq[8][4];
            {
                const __nv_bfloat16* qA = a.q + ((static_cast<long long>(b) * s.Hq + g * kG + hd) * s.R + (liveA ? tokA : 0)) * kD;
                const __nv_bfloat16* qB = a.q + ((static_cast<long long>(b) * s.Hq + g * kG + hd) * s.R + (liveB ? tokB : 0)) * kD;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    aq[ks][0] = liveA ? *reinterpret_cast<const uint32_t*>(qA + ks * 16 + 2 * t) : 0u;
                    aq[ks][1] = liveB ? *reinterpret_cast<const uint32_t*>(qB + ks * 16 + 2 * t) : 0u;
                    aq[ks][2] = liveA ? *reinterpret_cast<const uint32_t*>(qA + ks * 16 + 8 + 2 * t) : 0u;
                    aq[ks][3] = liveB ? *reinterpret_cast<const uint32_t*>(qB + ks * 16 + 8 + 2 * t) : 0u;
                }
            }
            float o[16][4];
#pragma unroll
            for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
            float mA = -INFINITY, mB = -INFINITY, dA = 0.f, dB = 0.f;      // running maximum / sum of the mixing logits
            const float sl2 = s.scale * kLog2e;
            bool dead = false;

            for (int j = 0; j < n_items; ++j) {
                const uint32_t it = n_item + j, st = it % kStages;
                if (!mbar_wait(&sm.full[st], (it / kStages) & 1)) {
                    if (lane == 0) { set_status(a.status, kDevTimeout); atomicExch(&sm.dead, 1); }
                    dead = true;
                    break;
                }
                const int c = item_chunk(j);
                const bool selected = j >= n_local;
                bool actA, actB;
                if (selected) {
                    const uint32_t mk = (sm.tokmask[c >> 1] >> ((c & 1) * 16)) & 0xffffu;
                    actA = liveA && ((mk >> tl0) & 1u);
                    actB = liveB && ((mk >> tl1) & 1u);
                } else {
                    actA = liveA && c >= lcA;
                    actB = liveB && c >= lcB;
                }
                if (__any_sync(kFullMask, actA || actB)) {
                    const uint32_t ks_addr = smem_u32(ring + st * kStride), vs_addr = ks_addr + 16384;
                    float sc[8][4];
                    qk_tile16(aq, ks_addr, lane, sc);
                    float lamA, lamB;
                    if (selected) {
                        // surrogate scores of the 16 rows against the chunk's landmark row: one more column of MMAs
                        // (column 0 of an 8-column tile; lanes 0..3 carry the landmark's elements)
                        const __nv_bfloat16* lmr = reinterpret_cast<const __nv_bfloat16*>(ring + st * kStride + 32768);
                        float dl[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            const uint32_t b0 = gq == 0 ? *reinterpret_cast<const uint32_t*>(lmr + ks * 16 + 2 * t) : 0u;
                            const uint32_t b1 = gq == 0 ? *reinterpret_cast<const uint32_t*>(lmr + ks * 16 + 8 + 2 * t) : 0u;
                            mma_bf16_16816(dl, aq[ks], b0, b1);
                        }
                        const float bb = a.bias ? a.bias[static_cast<long long>(pair) * s.C + c] : 0.f;
                        lamA = __shfl_sync(kFullMask, dl[0], lane & ~3) * s.scale + bb;
                        lamB = __shfl_sync(kFullMask, dl[2], lane & ~3) * s.scale + bb;
                    } else if (c == ci) {
                        // the tokens' own chunk: causal mask
                        const int limA = posA - c * kS, limB = posB - c * kS;
#pragma unroll
                        for (int nt = 0; nt < 8; ++nt) {
                            const int key = nt * 8 + 2 * t;
                            if (key > limA) sc[nt][0] = -INFINITY;
                            if (key + 1 > limA) sc[nt][1] = -INFINITY;
                            if (key > limB) sc[nt][2] = -INFINITY;
                            if (key + 1 > limB) sc[nt][3] = -INFINITY;
                        }
                        lamA = lamB = 0.f;
                    } else {
                        lamA = lamB = 0.f;
                    }
                    // the chunk's own softmax (Eq. HiLS weights, intra-chunk factor)
                    float xA = -INFINITY, xB = -INFINITY;
#pragma unroll
                    for (int nt = 0; nt < 8; ++nt) {
                        xA = fmaxf(xA, fmaxf(sc[nt][0], sc[nt][1]));
                        xB = fmaxf(xB, fmaxf(sc[nt][2], sc[nt][3]));
                    }
                    xA = fmaxf(xA, __shfl_xor_sync(kFullMask, xA, 1));
                    xB = fmaxf(xB, __shfl_xor_sync(kFullMask, xB, 1));
                    xA = fmaxf(xA, __shfl_xor_sync(kFullMask, xA, 2));
                    xB = fmaxf(xB, __shfl_xor_sync(kFullMask, xB, 2));
                    float zA = 0.f, zB = 0.f;
#pragma unroll
                    for (int nt = 0; nt < 8; ++nt) {
                        sc[nt][0] = exp2f((sc[nt][0] - xA) * sl2);
                        sc[nt][1] = exp2f((sc[nt][1] - xA) * sl2);
                        sc[nt][2] = exp2f((sc[nt][2] - xB) * sl2);
                        sc[nt][3] = exp2f((sc[nt][3] - xB) * sl2);
                        zA += sc[nt][0] + sc[nt][1];
                        zB += sc[nt][2] + sc[nt][3];
                    }
                    zA += __shfl_xor_sync(kFullMask, zA, 1);
                    zB += __shfl_xor_sync(kFullMask, zB, 1);
                    zA += __shfl_xor_sync(kFullMask, zA, 2);
                    zB += __shfl_xor_sync(kFullMask, zB, 2);
                    if (!selected) {
                        // a local chunk mixes with its exact log mass (Eq. chunk mass)
                        lamA = xA * s.scale + __logf(zA);
                        lamB = xB * s.scale + __logf(zB);
                    }
                    // running mix over the chunks (inter-chunk factor): rescale when the maximum moves
                    const float nA = actA ? fmaxf(mA, lamA) : mA, nB = actB ? fmaxf(mB, lamB) : mB;
                    const float fA = nA == mA ? 1.f : __expf(mA - nA), fB = nB == mB ? 1.f : __expf(mB - nB);
                    const float eA = actA ? __expf(lamA - nA) : 0.f, eB = actB ? __expf(lamB - nB) : 0.f;
                    dA = dA * fA + eA;
                    dB = dB * fB + eB;
                    mA = nA;
                    mB = nB;
                    if (__any_sync(kFullMask, fA != 1.f || fB != 1.f)) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) { o[i][0] *= fA; o[i][1] *= fA; o[i][2] *= fB; o[i][3] *= fB; }
                    }
                    const float wA = actA ? eA / zA : 0.f, wB = actB ? eB / zB : 0.f;
#pragma unroll
                    for (int nt = 0; nt < 8; ++nt) { sc[nt][0] *= wA; sc[nt][1] *= wA; sc[nt][2] *= wB; sc[nt][3] *= wB; }
                    pv_tile16(sc, vs_addr, lane, o);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.empty[st]);
            }
            if (!dead) {
                // every live token has attended at least its own position: the sums are positive
                const float iA = liveA ? 1.f / dA : 0.f, iB = liveB ? 1.f / dB : 0.f;
                __nv_bfloat16* oA = a.out + ((static_cast<long long>(b) * s.Hq + g * kG + hd) * s.R + (liveA ? tokA : 0)) * kD;
                __nv_bfloat16* oB = a.out + ((static_cast<long long>(b) * s.Hq + g * kG + hd) * s.R + (liveB ? tokB : 0)) * kD;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    if (liveA) *reinterpret_cast<uint32_t*>(oA + i * 8 + 2 * t) = pack_bf16(o[i][0] * iA, o[i][1] * iA);
                    if (liveB) *reinterpret_cast<uint32_t*>(oB + i * 8 + 2 * t) = pack_bf16(o[i][2] * iB, o[i][3] * iB);
                }
                if (t == 0) {
                    const long long lrow = static_cast<long long>(b) * s.Hq + g * kG + hd;
                    if (liveA) a.lse[lrow * s.R + tokA] = mA + __logf(dA);
                    if (liveB) a.lse[lrow * s.R + tokB] = mB + __logf(dB);
                }
            }
        }
        n_item += static_cast<uint32_t>(n_items);
        // the masks and the list belong to the next tile from here on; after a timeout every warp leaves
        __syncthreads();
        if (*reinterpret_cast<volatile int*>(&sm.dead)) break;
    }
}

}  // namespace

bool prefill_packed_supports(const Shape& s, int dtype) {
    return dtype == HILS_BF16 && !s.is_decode && s.d == kD && s.S == kS && s.G == kG && s.Hl == s.Hkv && s.K >= 1 &&
           s.K <= 32 && s.W >= 1 && (s.W - 1 + kS - 1) / kS + 1 <= kMaxLocal && s.pos0 % kM == 0 && s.C <= kMaxC &&
           (s.pos0 + s.R + kS - 1) / kS <= kMaxC && prefill_select_tc_supports(s) &&
           static_cast<long long>(s.B) * s.Hkv * s.T < (1ll << 31);
}

int launch_prefill_packed(const Shape& s, const Tensors& t, cudaStream_t stream) {
    const int pairs = s.B * s.Hkv;
    if (t.q_route) return HILS_ERR_UNSUPPORTED;      // (the mixing logits would need the routing query's scores)
    // selection: the tcgen05 scoring + top-K kernel
    const int rc = launch_prefill_select_tc(s, t.q, t.landmarks, t.bias, t.sel_idx, t.status, nullptr, 0, 0, stream);
    if (rc < 0) return rc;
    trace_mark("prefill_select", stream);
    CUtensorMap map_k, map_v;
    const uint64_t kv_rows = static_cast<uint64_t>(pairs) * s.T;
    if (!make_bf16_2d_map(&map_k, t.k, kv_rows, kD, 64, kS) || !make_bf16_2d_map(&map_v, t.v, kv_rows, kD, 64, kS))
        return HILS_ERR_CUDA;
    const size_t smem = kStages * (kStageBytes + 768) + sizeof(PkSmem) + 1024;
    static PerDeviceOnce attr_once;
    if (attr_once.pending()) {
        if (cudaFuncSetAttribute(prefill_packed_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem)) != cudaSuccess)
            return HILS_ERR_CUDA;
        attr_once.done();
    }
    PkArgs a;
    a.s = s;
    a.q = static_cast<const __nv_bfloat16*>(t.q);
    a.lm = static_cast<const __nv_bfloat16*>(t.landmarks);
    a.bias = t.bias;
    a.sel = t.sel_idx;
    a.out = static_cast<__nv_bfloat16*>(t.out);
    a.lse = t.lse;
    a.status = t.status;
    const long long n_tiles = static_cast<long long>(pairs) * ((s.R + kM - 1) / kM);
    const long long cap = 2ll * sm_count();
    prefill_packed_kernel<<<static_cast<unsigned>(n_tiles < cap ? n_tiles : cap), kThreads, smem, stream>>>(map_k, map_v, a);
    if (cudaGetLastError() != cudaSuccess) return HILS_ERR_CUDA;
    trace_mark("prefill_packed", stream);
    return 2;
}

}  // namespace hils
