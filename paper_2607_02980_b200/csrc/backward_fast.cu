// Backward of the HiLS operator for the benchmark shapes (bf16, d = 128, S = 64, four query heads per KV head,
// one landmark per KV head): chunk-major like the forward attend kernel, so that d k and d v of a chunk are
// accumulated on chip over all the queries that attend it.  Formulas: see backward.cu / the C header.
//
// The tiles of the forward's inverse index are reused: a tile is 32 (token, slot) entries x 4 heads = 128 query
// rows against one 64-key chunk.  A CTA of 8 warps walks a contiguous range of a query block's tiles.  K and V of
// the chunk arrive by TMA (128-byte swizzle), Q and dO rows by cp.async into the same swizzled layout.
//
// prefill_backward_tc_kernel (default): every product on the 5th-generation tensor cores, accumulators in tensor
//   memory.  S = Q K^T and T = dO V^T (K-major operands); warps 0-3 read one row each with tcgen05.ld, compute the
//   slot's softmax statistics thread-locally and write d S and W rows to shared memory as bf16; d Q = d S K (K read
//   MN-major); dK^T += Q^T d S and dV^T += dO^T W with both operands MN-major (the row tiles as they sit in shared
//   memory), accumulated in tensor memory over the tiles of a chunk.  Warps 4-7 read d Q of the previous tile out
//   beside the next tile's statistics (+ the landmark term, vector reductions into dq) and compute d landmark and
//   d bias; one thread issues the MMAs.
// prefill_backward_mma_kernel (HILS_BACKWARD_MMA_SYNC=1): the first version, every product on mma.sync with
//   ldmatrix operands: phase 1, warp = 16 rows: S, T, statistics with quad shuffles, d Q; phase 2, warp = 16 dims:
//   d K += d S^T Q, d V += W^T dO in registers across the tiles of a chunk.
#include <stdlib.h>

#include "internal.h"
#include "tma.cuh"

namespace hils {
namespace {

constexpr int kD = 128;
constexpr int kS = 64;
constexpr int kG = 4;
constexpr int kBfThreads = 256;
constexpr int kRows = 128;                 // rows of a tile: 32 entries x 4 heads, row = entry * 4 + head
constexpr int kKBytes = kS * kD * 2;       // 16 KB: two swizzled boxes of 64 dims x 64 keys
constexpr int kQBytes = kRows * kD * 2;    // 32 KB: two swizzled boxes of 64 dims x 128 rows
constexpr int kDsBytes = kRows * kS * 2;   // 16 KB: one swizzled box of 64 keys x 128 rows

struct BfArgs {
    Shape s;
    const __nv_bfloat16* q;
    const __nv_bfloat16* dout;
    const __nv_bfloat16* lm;
    const float* bias;
    const float* lse;
    const float* dsum;        // [B, Hq, R] dout . out
    const int* entries;
    const int4* tiles;
    const int* blk_range;     // {first tile of this query block, first tile of the next}
    float* dq;
    float* dk;
    float* dv;
    float* dlm;
    float* dbias;
    int* status;
    int i0;                   // first token of the query block
};

struct BfSmem {
    uint64_t kv_bar;
    float lmf[kD];            // the chunk's landmark
    float dlam[kRows];        // scale * d lambda of each row (0 for local-window and padding rows)
    // row tables of the tile in work and of the next one
    float row_lse[2][kRows];
    float row_dsum[2][kRows];
    int row_orow[2][kRows];   // (sequence, head, token) row of q / dout / dq, -1 = padding row
    int row_limit[2][kRows];  // last valid key column of the row (63 = whole chunk, -1 = none)
    int row_local[2][kRows];
    float bias_c;
    int abort_flag;
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void red_add_v2(float* p, float x, float y) {
    asm volatile("red.global.add.v2.f32 [%0], {%1, %2};" ::"l"(p), "f"(x), "f"(y) : "memory");
}

// Per-row dot products with dout: D = dout . out (one warp per row, 4 dims per lane).
__global__ void backward_dsum_kernel(const __nv_bfloat16* dout, const __nv_bfloat16* out, float* dsum, long long rows) {
    const long long row = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int lane = threadIdx.x & 31;
    const uint2 a = *reinterpret_cast<const uint2*>(dout + row * kD + lane * 4);
    const uint2 b = *reinterpret_cast<const uint2*>(out + row * kD + lane * 4);
    const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const float2 x = __bfloat1622float2(pa[i]), y = __bfloat1622float2(pb[i]);
        acc = fmaf(x.x, y.x, acc);
        acc = fmaf(x.y, y.y, acc);
    }
    acc = warp_sum(acc);
    if (lane == 0) dsum[row] = acc;
}

// C[16 x 64] = A[16 x 128] B^T.  A = rows r0 .. r0+15 of a [128 rows][128 dims] tile (two swizzled boxes of 64
// dims, kRows * 128 bytes apart), B = a [64 keys][128 dims] tile (two swizzled boxes, 8192 bytes apart).
// The 32-dim step is the outer loop so that consecutive MMAs go to different accumulators (the instructions are
// issued in program order; a chain on one accumulator would wait for each result).
__device__ __forceinline__ void rows_times_keys(uint32_t rows_addr, int r0, uint32_t keys_addr, int lane, float (&c)[8][4]) {
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f;
#pragma unroll
    for (int kp = 0; kp < 4; ++kp) {
        uint32_t a0[4], a1[4];
        {
            const int row = r0 + (lane & 7) + ((lane >> 3) & 1) * 8;
            const int dim = kp * 32 + (lane >> 4) * 8;
            ldmatrix_x4(rows_addr + (dim >> 6) * (kRows * 128) + swz128(row, (dim & 63) >> 3), a0[0], a0[1], a0[2], a0[3]);
            ldmatrix_x4(rows_addr + ((dim + 16) >> 6) * (kRows * 128) + swz128(row, ((dim + 16) & 63) >> 3), a1[0], a1[1],
                        a1[2], a1[3]);
        }
#pragma unroll
        for (int ng = 0; ng < 2; ++ng) {
            uint32_t b[4][4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = (ng * 4 + i) * 8 + (lane & 7);
                const int dim = kp * 32 + (lane >> 3) * 8;
                ldmatrix_x4(keys_addr + (dim >> 6) * 8192 + swz128(row, (dim & 63) >> 3), b[i][0], b[i][1], b[i][2], b[i][3]);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) mma_bf16_16816(c[ng * 4 + i], a0, b[i][0], b[i][1]);
#pragma unroll
            for (int i = 0; i < 4; ++i) mma_bf16_16816(c[ng * 4 + i], a1, b[i][2], b[i][3]);
        }
    }
}

__global__ void __launch_bounds__(kBfThreads, 1)
prefill_backward_mma_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                            const BfArgs a) {
    extern __shared__ uint8_t bf_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(bf_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* kbuf = base;
    uint8_t* vbuf = kbuf + kKBytes;
    uint8_t* qbuf0 = vbuf + kKBytes;             // [2][kQBytes]: the tile in work and the next one
    uint8_t* dobuf0 = qbuf0 + 2 * kQBytes;       // [2][kQBytes]
    uint8_t* dsbuf = dobuf0 + 2 * kQBytes;
    uint8_t* wbuf = dsbuf + kDsBytes;
    BfSmem& sm = *reinterpret_cast<BfSmem*>(wbuf + kDsBytes);

    const Shape& s = a.s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t4 = lane & 3;
    const int t_begin = a.blk_range[0], n_tiles = a.blk_range[1] - t_begin;
    const long long lo = t_begin + static_cast<long long>(blockIdx.x) * n_tiles / gridDim.x;
    const long long hi = t_begin + static_cast<long long>(blockIdx.x + 1) * n_tiles / gridDim.x;

    if (tid == 0) {
        mbar_init(&sm.kv_bar, 1);
        mbar_fence_init();
        sm.abort_flag = 0;
        tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v);
    }
    __syncthreads();

    const uint32_t k_addr = smem_u32(kbuf), v_addr = smem_u32(vbuf);
    const uint32_t ds_addr = smem_u32(dsbuf), w_addr = smem_u32(wbuf);
    uint32_t kv_phase = 0;
    int cur_pair = -1, cur_c = -1;
    float dk_acc[4][2][4], dv_acc[4][2][4];
    float lm_acc = 0.f, bias_acc = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int x = 0; x < 4; ++x) dk_acc[i][j][x] = dv_acc[i][j][x] = 0.f;

    // adds the finished chunk's register accumulators to dk, dv, dlandmarks, dbias and clears them
    auto flush = [&]() {
        if (cur_pair < 0) return;
        const int b = cur_pair / s.Hkv, gk = cur_pair % s.Hkv;
        const long long kvrow0 = static_cast<long long>(cur_pair) * s.T;
#pragma unroll
        for (int mt = 0; mt < 4; ++mt)
#pragma unroll
            for (int n2 = 0; n2 < 2; ++n2) {
                const int dim = warp * 16 + n2 * 8 + 2 * t4;
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int key = cur_c * kS + mt * 16 + g + hh * 8;
                    if (key < s.T) {
                        red_add_v2(a.dk + (kvrow0 + key) * kD + dim, dk_acc[mt][n2][2 * hh], dk_acc[mt][n2][2 * hh + 1]);
                        red_add_v2(a.dv + (kvrow0 + key) * kD + dim, dv_acc[mt][n2][2 * hh], dv_acc[mt][n2][2 * hh + 1]);
                    }
                    dk_acc[mt][n2][2 * hh] = dk_acc[mt][n2][2 * hh + 1] = 0.f;
                    dv_acc[mt][n2][2 * hh] = dv_acc[mt][n2][2 * hh + 1] = 0.f;
                }
            }
        lm_acc += __shfl_xor_sync(kFullMask, lm_acc, 16);
        if (cur_c < s.C) {
            const long long lrow = (static_cast<long long>(b) * s.Hl + gk) * s.C + cur_c;
            if (lane < 16) atomicAdd(a.dlm + lrow * kD + warp * 16 + lane, lm_acc);
            if (warp == 0 && lane == 0 && a.dbias) atomicAdd(a.dbias + lrow, bias_acc / s.scale);
        }
        lm_acc = 0.f;
        bias_acc = 0.f;
    };

    // Requests the chunk's K and V (TMA, thread 0) and reads its landmark and bias (threads 128..255).  Called when
    // nobody reads the previous chunk's copies any more.
    auto issue_chunk = [&](int pair, int c) {
        const int b = pair / s.Hkv, gk = pair % s.Hkv;
        if (tid == 0) {
            const int row = pair * s.T + c * kS;
            mbar_expect_tx(&sm.kv_bar, 2 * kKBytes);
            tma_load_2d(kbuf, &map_k, &sm.kv_bar, 0, row);
            tma_load_2d(kbuf + 8192, &map_k, &sm.kv_bar, 64, row);
            tma_load_2d(vbuf, &map_v, &sm.kv_bar, 0, row);
            tma_load_2d(vbuf + 8192, &map_v, &sm.kv_bar, 64, row);
        } else if (tid >= kRows) {
            const int x = tid - kRows;
            const long long lrow = (static_cast<long long>(b) * s.Hl + gk) * s.C + c;
            sm.lmf[x] = c < s.C ? __bfloat162float(a.lm[lrow * kD + x]) : 0.f;
            if (x == 0) sm.bias_c = (a.bias && c < s.C) ? a.bias[lrow] : 0.f;
        }
    };
    // Starts the gather of a tile's Q and dO rows into buffer `par` (thread -> row tid / 2, 64-dim half tid & 1;
    // padding rows are zero) and returns what the row table needs; store_row() writes it once the loads are back.
    struct RowInfo { int orow, limit, local; float lse, dsum; };
    // entry of this thread's row in a tile (read two tiles ahead of its use, so that no tile waits for it)
    auto load_entry = [&](const int4 rec) { return (tid >> 3) < rec.w ? a.entries[rec.z + (tid >> 3)] : 0; };
    auto issue_tile = [&](const int4 rec, int ent, int par) {
        const int pair = rec.x, c = rec.y, ntok = rec.w;
        const int b = pair / s.Hkv, gk = pair % s.Hkv;
        const int row = tid >> 1, half = tid & 1, e = row >> 2, h = row & 3;
        RowInfo ri{-1, -1, 0, 0.f, 0.f};
        uint8_t* qb = qbuf0 + par * kQBytes + half * (kRows * 128);
        uint8_t* db = dobuf0 + par * kQBytes + half * (kRows * 128);
        if (e < ntok) {
            const int tok = a.i0 + (ent >> 8), slot = ent & 255;
            ri.orow = (b * s.Hq + gk * kG + h) * s.R + tok;
            ri.local = slot >= s.K ? 1 : 0;
            ri.limit = ri.local ? min(kS - 1, s.pos0 + tok - c * kS) : kS - 1;
            const __nv_bfloat16* qs = a.q + static_cast<long long>(ri.orow) * kD + half * 64;
            const __nv_bfloat16* ds = a.dout + static_cast<long long>(ri.orow) * kD + half * 64;
            const uint32_t qa = smem_u32(qb), da = smem_u32(db);
#pragma unroll
            for (int p = 0; p < 8; ++p) {
                cp_async16(qa + swz128(row, p), qs + p * 8);
                cp_async16(da + swz128(row, p), ds + p * 8);
            }
            if (half == 0) {
                ri.lse = a.lse[ri.orow];
                ri.dsum = a.dsum[ri.orow];
            }
        } else {
#pragma unroll
            for (int p = 0; p < 8; ++p) {
                *reinterpret_cast<uint4*>(qb + swz128(row, p)) = make_uint4(0u, 0u, 0u, 0u);
                *reinterpret_cast<uint4*>(db + swz128(row, p)) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        return ri;
    };
    auto store_row = [&](const RowInfo& ri, int par) {
        if ((tid & 1) == 0) {
            const int row = tid >> 1;
            sm.row_orow[par][row] = ri.orow;
            sm.row_limit[par][row] = ri.limit;
            sm.row_local[par][row] = ri.local;
            sm.row_lse[par][row] = ri.lse;
            sm.row_dsum[par][row] = ri.dsum;
        }
    };

    const int4 no_tile = make_int4(-1, -1, 0, 0);
    int4 rec = no_tile, nrec = no_tile, n2rec = no_tile;       // this tile, the next one, the one after
    int nent = 0;                                              // this thread's entry in the next tile
    bool kv_issued = false;
    if (lo < hi) {
        rec = a.tiles[lo];
        if (lo + 1 < hi) nrec = a.tiles[lo + 1];
        if (lo + 2 < hi) n2rec = a.tiles[lo + 2];
        issue_chunk(rec.x, rec.y);
        kv_issued = true;
        store_row(issue_tile(rec, load_entry(rec), 0), 0);
        nent = load_entry(nrec);
    }
    for (long long tile = lo; tile < hi; ++tile) {
        const int par = static_cast<int>(tile - lo) & 1;
        const int pair = rec.x, c = rec.y;
        cur_pair = pair;
        cur_c = c;
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        if (kv_issued) {
            if (!mbar_wait(&sm.kv_bar, kv_phase)) {
                sm.abort_flag = 1;
                if (lane == 0) set_status(a.status, kDevTimeout);
            }
            kv_phase ^= 1u;
            kv_issued = false;
        }
        __syncthreads();                        // this tile's Q, dO, row table, K, V, landmark are in shared memory;
                                                // the previous tile's readers are done with the other buffers
        if (sm.abort_flag) break;
        // the next tile's rows start to arrive while this one is computed
        const bool has_next = tile + 1 < hi;
        RowInfo nri{-1, -1, 0, 0.f, 0.f};
        if (has_next) nri = issue_tile(nrec, nent, par ^ 1);
        // metadata of the tiles after the next: in registers by the time they are needed
        const int n2ent = load_entry(n2rec);
        const int4 n3rec = tile + 3 < hi ? a.tiles[tile + 3] : no_tile;
        const bool next_new = has_next && (nrec.x != pair || nrec.y != c);
        const uint8_t* qbuf = qbuf0 + par * kQBytes;
        const uint32_t q_addr = smem_u32(qbuf), do_addr = smem_u32(dobuf0 + par * kQBytes);

        // ------------------------------------------------------------------ phase 1: rows 16 warp .. 16 warp + 15
        const int r0 = warp * 16;
        const int rA = r0 + g, rB = rA + 8;
        float lamA, lamB;
        {   // surrogate score of each row: two lanes per row, 64 dims each
            const int row = r0 + (lane >> 1), half = lane & 1;
            float acc = 0.f;
#pragma unroll
            for (int p = 0; p < 8; ++p) {
                const uint4 v = *reinterpret_cast<const uint4*>(qbuf + half * (kRows * 128) + swz128(row, p));
                const __nv_bfloat162* pv = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 x = __bfloat1622float2(pv[i]);
                    acc = fmaf(x.x, sm.lmf[half * 64 + p * 8 + 2 * i], acc);
                    acc = fmaf(x.y, sm.lmf[half * 64 + p * 8 + 2 * i + 1], acc);
                }
            }
            acc += __shfl_xor_sync(kFullMask, acc, 1);
            const float lam = acc * s.scale + sm.bias_c;
            lamA = __shfl_sync(kFullMask, lam, 2 * g);
            lamB = __shfl_sync(kFullMask, lam, 2 * (g + 8));
        }

        float sc[8][4], tc[8][4];
        rows_times_keys(q_addr, r0, k_addr, lane, sc);
        rows_times_keys(do_addr, r0, v_addr, lane, tc);

        float dlam2[2];
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int row = hh ? rB : rA;
            const int limit = sm.row_limit[par][row];
            const bool local = sm.row_local[par][row] != 0;
            const float lse = sm.row_lse[par][row], dsum = sm.row_dsum[par][row], lam = hh ? lamB : lamA;
            // the slot's own softmax statistics: computed for every row (the quad shuffles must not sit in a
            // branch that differs between the rows of a warp), used by the rows of selected chunks only
            float m = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) m = fmaxf(m, fmaxf(sc[nt][2 * hh], sc[nt][2 * hh + 1]));
            m = fmaxf(m, __shfl_xor_sync(kFullMask, m, 1));
            m = fmaxf(m, __shfl_xor_sync(kFullMask, m, 2));
            m *= s.scale;
            float Z = 0.f, gt = 0.f;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const float e = __expf(sc[nt][2 * hh + i] * s.scale - m);
                    Z += e;
                    gt = fmaf(e, tc[nt][2 * hh + i], gt);
                }
            Z += __shfl_xor_sync(kFullMask, Z, 1);
            Z += __shfl_xor_sync(kFullMask, Z, 2);
            gt += __shfl_xor_sync(kFullMask, gt, 1);
            gt += __shfl_xor_sync(kFullMask, gt, 2);
            float shift = lse, sub = dsum, dl = 0.f;
            if (!local) {
                const float gc = gt / Z;
                const float alpha = __expf(lam - lse);
                shift = m + __logf(Z) - (lam - lse);
                sub = gc;
                dl = limit >= 0 ? alpha * (gc - dsum) * s.scale : 0.f;
            }
            dlam2[hh] = dl;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int col = nt * 8 + 2 * t4 + i;
                    const float w = col <= limit ? __expf(sc[nt][2 * hh + i] * s.scale - shift) : 0.f;
                    sc[nt][2 * hh + i] = w * (tc[nt][2 * hh + i] - sub) * s.scale;     // d s_j (times scale)
                    tc[nt][2 * hh + i] = w;                                           // w_j
                }
        }
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            *reinterpret_cast<uint32_t*>(dsbuf + swz128(rA, nt) + 4 * t4) = pack_bf16(sc[nt][0], sc[nt][1]);
            *reinterpret_cast<uint32_t*>(dsbuf + swz128(rB, nt) + 4 * t4) = pack_bf16(sc[nt][2], sc[nt][3]);
            *reinterpret_cast<uint32_t*>(wbuf + swz128(rA, nt) + 4 * t4) = pack_bf16(tc[nt][0], tc[nt][1]);
            *reinterpret_cast<uint32_t*>(wbuf + swz128(rB, nt) + 4 * t4) = pack_bf16(tc[nt][2], tc[nt][3]);
        }
        if (t4 == 0) {
            sm.dlam[rA] = dlam2[0];
            sm.dlam[rB] = dlam2[1];
        }

        {   // d Q = d S K + d lambda k' for the warp's 16 rows
            float o[16][4];
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                const uint32_t af[4] = {pack_bf16(sc[2 * kk][0], sc[2 * kk][1]), pack_bf16(sc[2 * kk][2], sc[2 * kk][3]),
                                        pack_bf16(sc[2 * kk + 1][0], sc[2 * kk + 1][1]),
                                        pack_bf16(sc[2 * kk + 1][2], sc[2 * kk + 1][3])};
#pragma unroll
                for (int dp = 0; dp < 8; ++dp) {
                    const int mat = lane >> 3;
                    const int row = kk * 16 + (mat & 1) * 8 + (lane & 7);
                    const int dim = dp * 16 + (mat >> 1) * 8;
                    uint32_t r0v, r1v, r2v, r3v;
                    ldmatrix_x4_trans(k_addr + (dim >> 6) * 8192 + swz128(row, (dim & 63) >> 3), r0v, r1v, r2v, r3v);
                    mma_bf16_16816(o[2 * dp], af, r0v, r1v);
                    mma_bf16_16816(o[2 * dp + 1], af, r2v, r3v);
                }
            }
            const int orowA = sm.row_orow[par][rA], orowB = sm.row_orow[par][rB];
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) {
                const int col = nt * 8 + 2 * t4;
                const float l0 = sm.lmf[col], l1 = sm.lmf[col + 1];
                if (orowA >= 0)
                    red_add_v2(a.dq + static_cast<long long>(orowA) * kD + col, fmaf(dlam2[0], l0, o[nt][0]),
                               fmaf(dlam2[0], l1, o[nt][1]));
                if (orowB >= 0)
                    red_add_v2(a.dq + static_cast<long long>(orowB) * kD + col, fmaf(dlam2[1], l0, o[nt][2]),
                               fmaf(dlam2[1], l1, o[nt][3]));
            }
        }
        if (has_next) store_row(nri, par ^ 1);
        __syncthreads();                        // d S, W and d lambda of all 128 rows are in shared memory
        if (next_new) {                         // K, V and the landmark are not read in phase 2: fetch the next chunk's
            issue_chunk(nrec.x, nrec.y);
            kv_issued = true;
        }

        // ------------------------------------------------------------------ phase 2: dims 16 warp .. 16 warp + 15
#pragma unroll 2
        for (int ks = 0; ks < 8; ++ks) {
            const int mat = lane >> 3;
            uint32_t bq[4], bo[4];
            {
                const int row = ks * 16 + (mat & 1) * 8 + (lane & 7);
                const int dim = warp * 16 + (mat >> 1) * 8;
                const uint32_t off = (dim >> 6) * (kRows * 128) + swz128(row, (dim & 63) >> 3);
                ldmatrix_x4_trans(q_addr + off, bq[0], bq[1], bq[2], bq[3]);
                ldmatrix_x4_trans(do_addr + off, bo[0], bo[1], bo[2], bo[3]);
            }
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) {
                const int row = ks * 16 + (mat >> 1) * 8 + (lane & 7);
                const uint32_t off = swz128(row, 2 * mt + (mat & 1));
                uint32_t ad[4], aw[4];
                ldmatrix_x4_trans(ds_addr + off, ad[0], ad[1], ad[2], ad[3]);
                ldmatrix_x4_trans(w_addr + off, aw[0], aw[1], aw[2], aw[3]);
                mma_bf16_16816(dk_acc[mt][0], ad, bq[0], bq[1]);
                mma_bf16_16816(dk_acc[mt][1], ad, bq[2], bq[3]);
                mma_bf16_16816(dv_acc[mt][0], aw, bo[0], bo[1]);
                mma_bf16_16816(dv_acc[mt][1], aw, bo[2], bo[3]);
            }
        }
        {   // d landmark: sum over rows of (scale d lambda_r) q_r, lane -> (dim, half of the rows)
            const int dim = warp * 16 + (lane & 15), half = lane >> 4;
            const uint8_t* col = qbuf + (dim >> 6) * (kRows * 128) + (dim & 7) * 2;
            const int piece = (dim & 63) >> 3;
            float acc = 0.f;
#pragma unroll 8
            for (int r = half * 64; r < half * 64 + 64; ++r) {
                const float dl = sm.dlam[r];
                const __nv_bfloat16 x = *reinterpret_cast<const __nv_bfloat16*>(col + swz128(r, piece));
                acc = fmaf(dl, __bfloat162float(x), acc);
            }
            lm_acc += acc;
            if (warp == 0) {
                const float v = sm.dlam[lane] + sm.dlam[lane + 32] + sm.dlam[lane + 64] + sm.dlam[lane + 96];
                bias_acc += warp_sum(v);
            }
        }
        if (!has_next || next_new) flush();
        rec = nrec;
        nrec = n2rec;
        nent = n2ent;
        n2rec = n3rec;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

struct BtSmem {               // shared state of the tcgen05 variant
    uint64_t kv_bar, st_bar, dq_bar, p2_bar;
    uint32_t tmem_base;
    alignas(16) float lmf[2][kD];   // the landmark of the chunk in work and of the next one
    float bias_c[2];
    float dlam[kRows];
    float row_lse[2][kRows];
    float row_dsum[2][kRows];
    int row_orow[2][kRows];
    int row_limit[2][kRows];
    int row_local[2][kRows];
    int abort_flag;
};
constexpr uint32_t kUmmaAMnMajor = 1u << 15;     // instruction-descriptor bit: A operand is MN-major
__device__ __forceinline__ void red_add_f32(float* p, float x) {
    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(p), "f"(x) : "memory");
}
__device__ __forceinline__ void red_add_v4(float* p, float x, float y, float z, float w) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(x), "f"(y), "f"(z), "f"(w) : "memory");
}

__global__ void __launch_bounds__(kBfThreads, 1)
prefill_backward_tc_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                            const BfArgs a) {
    extern __shared__ uint8_t bf_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(bf_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* kbuf = base;
    uint8_t* vbuf = kbuf + kKBytes;
    uint8_t* qbuf0 = vbuf + kKBytes;             // [2][kQBytes]: the tile in work and the next one
    uint8_t* dobuf0 = qbuf0 + 2 * kQBytes;       // [2][kQBytes]
    uint8_t* dsbuf = dobuf0 + 2 * kQBytes;
    uint8_t* wbuf = dsbuf + kDsBytes;
    BtSmem& sm = *reinterpret_cast<BtSmem*>(wbuf + kDsBytes);

    const Shape& s = a.s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t4 = lane & 3;
    const int t_begin = a.blk_range[0], n_tiles = a.blk_range[1] - t_begin;
    const long long lo = t_begin + static_cast<long long>(blockIdx.x) * n_tiles / gridDim.x;
    const long long hi = t_begin + static_cast<long long>(blockIdx.x + 1) * n_tiles / gridDim.x;

    if (tid == 0) {
        mbar_init(&sm.kv_bar, 1);
        mbar_init(&sm.st_bar, 1);
        mbar_init(&sm.dq_bar, 1);
        mbar_init(&sm.p2_bar, 1);
        mbar_fence_init();
        sm.abort_flag = 0;
        tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v);
    }
    if (warp == 0) tmem_alloc(&sm.tmem_base, 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = sm.tmem_base;
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);     // this warp's 32 rows
    // tensor-memory columns: S = Q K^T at 0..63, T = dO V^T at 64..127, dQ at 128..255,
    // dK^T (dims x keys) at 256..319, dV^T at 320..383
    uint32_t st_phase = 0, dq_phase = 0, p2_phase = 0;
    bool run_acc = false;                              // the chunk's dK^T / dV^T accumulators hold earlier tiles
    int cpar = 0;                                      // which copy of the landmark / bias belongs to the chunk in work
    bool st_issued = false;                            // S / T MMAs of the tile at the loop top were issued a tile early
    // read-out of d Q one tile late (warps 4-7), beside the next tile's row statistics (warps 0-3)
    int ro_orow = -1, ro_cpar = 0;
    float ro_dl = 0.f;
    bool ro_pending = false;
    auto read_out = [&]() {
        // thread = row (warps 4-7): d Q row from tensor memory + d lambda k', added to dq
        if (!mbar_wait(&sm.dq_bar, dq_phase ^ 1u)) {
            sm.abort_flag = 1;
            if (lane == 0) set_status(a.status, kDevTimeout);
        }
        tc_fence_after_sync();
        float o0[64], o1[64];
        tmem_ld64x2(t_lane + 128, t_lane + 192, o0, o1);
        if (ro_orow >= 0) {
            float* dst = a.dq + static_cast<long long>(ro_orow) * kD;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float* l = &sm.lmf[ro_cpar][4 * i];
                red_add_v4(dst + 4 * i, fmaf(ro_dl, l[0], o0[4 * i]), fmaf(ro_dl, l[1], o0[4 * i + 1]),
                           fmaf(ro_dl, l[2], o0[4 * i + 2]), fmaf(ro_dl, l[3], o0[4 * i + 3]));
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float* l = &sm.lmf[ro_cpar][64 + 4 * i];
                red_add_v4(dst + 64 + 4 * i, fmaf(ro_dl, l[0], o1[4 * i]), fmaf(ro_dl, l[1], o1[4 * i + 1]),
                           fmaf(ro_dl, l[2], o1[4 * i + 2]), fmaf(ro_dl, l[3], o1[4 * i + 3]));
            }
        }
        tc_fence_before_sync();
    };

    const uint32_t k_addr = smem_u32(kbuf), v_addr = smem_u32(vbuf);
    const uint64_t dk0 = umma_desc_k128(k_addr), dv0 = umma_desc_k128(v_addr);                 // K, V as K-major operands
    const uint64_t dkmn0 = umma_desc_mn128(k_addr, 8192u, 1024u);                               // K as an MN-major operand
    const uint64_t dds0 = umma_desc_k128(smem_u32(dsbuf));                                      // d S, K-major (d Q)
    const uint64_t ddsmn0 = umma_desc_mn128(smem_u32(dsbuf), 8192u, 1024u);                     // d S, W MN-major (dK, dV)
    const uint64_t dwmn0 = umma_desc_mn128(smem_u32(wbuf), 8192u, 1024u);
    const uint32_t ds_addr = smem_u32(dsbuf), w_addr = smem_u32(wbuf);
    uint32_t kv_phase = 0;
    int cur_pair = -1, cur_c = -1;
    float lm_acc = 0.f, bias_acc = 0.f;

    // Adds the finished chunk's accumulators to dk, dv, dlandmarks, dbias.  dK^T and dV^T sit in tensor memory with a
    // lane per dimension: warps 0-3 read dK^T, warps 4-7 dV^T (64 keys each), a reduction of 32 consecutive
    // dimensions per key and warp.  Called by every thread after the chunk's last MMAs were issued.
    auto flush = [&]() {
        if (cur_pair < 0) return;
        const int b = cur_pair / s.Hkv, gk = cur_pair % s.Hkv;
        const long long kvrow0 = static_cast<long long>(cur_pair) * s.T;
        if (!mbar_wait(&sm.p2_bar, p2_phase ^ 1u)) {
            sm.abort_flag = 1;
            if (lane == 0) set_status(a.status, kDevTimeout);
        }
        tc_fence_after_sync();
        {
            float acc[64];
            tmem_ld64(t_lane + 256 + (warp >= 4 ? 64 : 0), acc);
            float* dst = (warp >= 4 ? a.dv : a.dk) + kvrow0 * kD + (warp & 3) * 32 + lane;
#pragma unroll
            for (int j = 0; j < 64; ++j) {
                const int key = cur_c * kS + j;
                if (key < s.T) red_add_f32(dst + static_cast<long long>(key) * kD, acc[j]);
            }
        }
        tc_fence_before_sync();
        run_acc = false;
        if (cur_c < s.C && warp >= 4) {
            const long long lrow = (static_cast<long long>(b) * s.Hl + gk) * s.C + cur_c;
            atomicAdd(a.dlm + lrow * kD + (warp - 4) * 32 + lane, lm_acc);
            if (warp == 4 && lane == 0 && a.dbias) atomicAdd(a.dbias + lrow, bias_acc / s.scale);
        }
        lm_acc = 0.f;
        bias_acc = 0.f;
    };

    // Requests the chunk's K and V (TMA, thread 0) and reads its landmark and bias (threads 128..255).  Called when
    // nobody reads the previous chunk's copies any more.
    auto issue_chunk = [&](int pair, int c, int cp) {
        const int b = pair / s.Hkv, gk = pair % s.Hkv;
        if (tid == kRows) {
            const int row = pair * s.T + c * kS;
            mbar_expect_tx(&sm.kv_bar, 2 * kKBytes);
            tma_load_2d(kbuf, &map_k, &sm.kv_bar, 0, row);
            tma_load_2d(kbuf + 8192, &map_k, &sm.kv_bar, 64, row);
            tma_load_2d(vbuf, &map_v, &sm.kv_bar, 0, row);
            tma_load_2d(vbuf + 8192, &map_v, &sm.kv_bar, 64, row);
        }
        if (tid >= kRows) {
            const int x = tid - kRows;
            const long long lrow = (static_cast<long long>(b) * s.Hl + gk) * s.C + c;
            sm.lmf[cp][x] = c < s.C ? __bfloat162float(a.lm[lrow * kD + x]) : 0.f;
            if (x == 0) sm.bias_c[cp] = (a.bias && c < s.C) ? a.bias[lrow] : 0.f;
        }
    };
    // Starts the gather of a tile's Q and dO rows into buffer `par` (thread -> row tid / 2, 64-dim half tid & 1;
    // padding rows are zero) and returns what the row table needs; store_row() writes it once the loads are back.
    struct RowInfo { int orow, limit, local; float lse, dsum; };
    // entry of this thread's row in a tile (read two tiles ahead of its use, so that no tile waits for it)
    auto load_entry = [&](const int4 rec) { return (tid >> 3) < rec.w ? a.entries[rec.z + (tid >> 3)] : 0; };
    // Gather of a tile's Q and dO rows.  Eight consecutive lanes fetch the eight 16-byte pieces of one 128-byte
    // half row, so every request covers whole lines; a group of eight lanes owns one entry = its four heads' rows.
    // The copies are requested in four parts (head g in part g), spread over the computation of the tile before.
    struct Gather { const __nv_bfloat16* qs; const __nv_bfloat16* ds; uint32_t qa, da; int row0; bool valid; };
    auto gather_part = [&](const Gather& gt, int g) {
        if (gt.valid) {
            const int row = gt.row0 + g, pc = tid & 7;
            const long long src = static_cast<long long>(g) * s.R * kD;          // head g of the entry's token
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                cp_async16(gt.qa + half * (kRows * 128) + swz128(row, pc), gt.qs + src + half * 64);
                cp_async16(gt.da + half * (kRows * 128) + swz128(row, pc), gt.ds + src + half * 64);
            }
        }
    };
    auto issue_tile = [&](const int4 rec, int ent, int par, Gather* defer = nullptr) {
        const int pair = rec.x, c = rec.y, ntok = rec.w;
        const int b = pair / s.Hkv, gk = pair % s.Hkv;
        const int row = tid >> 1, e = tid >> 3, h = row & 3;               // e = the entry of row tid / 2 as well
        RowInfo ri{-1, -1, 0, 0.f, 0.f};
        uint8_t* qb = qbuf0 + par * kQBytes;
        uint8_t* db = dobuf0 + par * kQBytes;
        if (e < ntok) {
            const int tok = a.i0 + (ent >> 8), slot = ent & 255;
            const int orow0 = (b * s.Hq + gk * kG) * s.R + tok;            // head 0 of the entry
            ri.orow = orow0 + h * s.R;
            ri.local = slot >= s.K ? 1 : 0;
            ri.limit = ri.local ? min(kS - 1, s.pos0 + tok - c * kS) : kS - 1;
            const Gather gt{a.q + static_cast<long long>(orow0) * kD + (tid & 7) * 8,
                            a.dout + static_cast<long long>(orow0) * kD + (tid & 7) * 8, smem_u32(qb), smem_u32(db), e * 4, true};
            if (defer) {
                *defer = gt;
                gather_part(gt, 0);
            } else {
#pragma unroll
                for (int g4 = 0; g4 < 4; ++g4) gather_part(gt, g4);
            }
            if ((tid & 1) == 0) {
                ri.lse = a.lse[ri.orow];
                ri.dsum = a.dsum[ri.orow];
            }
        } else {
            // padding entry: its four rows are zero
#pragma unroll
            for (int g4 = 0; g4 < 4; ++g4)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    *reinterpret_cast<uint4*>(qb + half * (kRows * 128) + swz128(e * 4 + g4, tid & 7)) = make_uint4(0u, 0u, 0u, 0u);
                    *reinterpret_cast<uint4*>(db + half * (kRows * 128) + swz128(e * 4 + g4, tid & 7)) = make_uint4(0u, 0u, 0u, 0u);
                }
        }
        if (!defer) asm volatile("cp.async.commit_group;" ::: "memory");
        return ri;
    };
    auto store_row = [&](const RowInfo& ri, int par) {
        if ((tid & 1) == 0) {
            const int row = tid >> 1;
            sm.row_orow[par][row] = ri.orow;
            sm.row_limit[par][row] = ri.limit;
            sm.row_local[par][row] = ri.local;
            sm.row_lse[par][row] = ri.lse;
            sm.row_dsum[par][row] = ri.dsum;
        }
    };

    const int4 no_tile = make_int4(-1, -1, 0, 0);
    int4 rec = no_tile, nrec = no_tile, n2rec = no_tile;       // this tile, the next one, the one after
    int nent = 0;                                              // this thread's entry in the next tile
    bool kv_issued = false;
    if (lo < hi) {
        rec = a.tiles[lo];
        if (lo + 1 < hi) nrec = a.tiles[lo + 1];
        if (lo + 2 < hi) n2rec = a.tiles[lo + 2];
        issue_chunk(rec.x, rec.y, 0);
        kv_issued = true;
        store_row(issue_tile(rec, load_entry(rec), 0), 0);
        nent = load_entry(nrec);
    }
    for (long long tile = lo; tile < hi; ++tile) {
        const int par = static_cast<int>(tile - lo) & 1;
        const int pair = rec.x, c = rec.y;
        cur_pair = pair;
        cur_c = c;
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        fence_proxy_async_smem();                   // the gathered rows are read by the tensor cores (async proxy)
        // the previous tile's dK / dV MMAs read its Q, dO rows and d S, W: all of them are overwritten from here on
        if (tile > lo && !mbar_wait(&sm.p2_bar, p2_phase ^ 1u)) {
            sm.abort_flag = 1;
            if (lane == 0) set_status(a.status, kDevTimeout);
        }
        if (kv_issued) {
            if (!mbar_wait(&sm.kv_bar, kv_phase)) {
                sm.abort_flag = 1;
                if (lane == 0) set_status(a.status, kDevTimeout);
            }
            kv_phase ^= 1u;
            kv_issued = false;
        }
        __syncthreads();                        // this tile's Q, dO, row table, K, V, landmark are in shared memory;
                                                // the previous tile's readers are done with the other buffers
        if (sm.abort_flag) break;
        // the next tile's rows start to arrive while this one is computed
        const bool has_next = tile + 1 < hi;
        RowInfo nri{-1, -1, 0, 0.f, 0.f};
        Gather gth{nullptr, nullptr, 0u, 0u, 0, false};
        if (has_next) nri = issue_tile(nrec, nent, par ^ 1, &gth);
        // metadata of the tiles after the next: in registers by the time they are needed
        const int n2ent = load_entry(n2rec);
        const int4 n3rec = tile + 3 < hi ? a.tiles[tile + 3] : no_tile;
        const bool next_new = has_next && (nrec.x != pair || nrec.y != c);
        const uint8_t* qbuf = qbuf0 + par * kQBytes;
        const uint32_t q_addr = smem_u32(qbuf), do_addr = smem_u32(dobuf0 + par * kQBytes);

        // ------------------------------------------------------------------ S = Q K^T and T = dO V^T on tcgen05
        // (a descriptor's start address is its low field in units of 16 bytes: a later k-step is the first one's
        // descriptor plus the byte offset / 16; nothing here comes near a carry out of the field)
        auto issue_st = [&](uint32_t qa, uint32_t da) {          // one thread: S = Q K^T, T = dO V^T
            constexpr uint32_t idesc_st = umma_idesc_bf16(kRows, kS);
            tc_fence_after_sync();
            const uint64_t dq0 = umma_desc_k128(qa), dd0 = umma_desc_k128(da);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                umma_bf16(tmem_base, dq0 + (((ks >> 2) * (kRows * 128) + (ks & 3) * 32) >> 4),
                          dk0 + (((ks >> 2) * 8192 + (ks & 3) * 32) >> 4), idesc_st, ks > 0 ? 1u : 0u);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                umma_bf16(tmem_base + 64, dd0 + (((ks >> 2) * (kRows * 128) + (ks & 3) * 32) >> 4),
                          dv0 + (((ks >> 2) * 8192 + (ks & 3) * 32) >> 4), idesc_st, ks > 0 ? 1u : 0u);
            umma_commit(&sm.st_bar);
        };
        if (tid == 0 && !st_issued) issue_st(q_addr, do_addr);
        // the previous tile's d Q leaves tensor memory while this tile's statistics are computed
        if (warp >= 4) {
            gather_part(gth, 1);
            if (ro_pending) read_out();
            gather_part(gth, 2);
            gather_part(gth, 3);
        }
        ro_pending = false;
        // ------------------------------------------------------------------ phase 1: warps 0-3, one row per thread
        if (warp < 4) {
            const int row = tid;
            const int limit = sm.row_limit[par][row];
            const bool local = sm.row_local[par][row] != 0;
            const float lse = sm.row_lse[par][row], dsum = sm.row_dsum[par][row];
            // surrogate score of the row (its own Q row against the landmark) while the MMAs run
            float lam = 0.f, lam2 = 0.f;
#pragma unroll
            for (int half = 0; half < 2; ++half)
#pragma unroll
                for (int pc = 0; pc < 8; ++pc) {
                    const uint4 v = *reinterpret_cast<const uint4*>(qbuf + half * (kRows * 128) + swz128(row, pc));
                    const __nv_bfloat162* pv = reinterpret_cast<const __nv_bfloat162*>(&v);
                    const float4 l0 = *reinterpret_cast<const float4*>(&sm.lmf[cpar][half * 64 + pc * 8]);
                    const float4 l1 = *reinterpret_cast<const float4*>(&sm.lmf[cpar][half * 64 + pc * 8 + 4]);
                    const float2 x0 = __bfloat1622float2(pv[0]), x1 = __bfloat1622float2(pv[1]);
                    const float2 x2 = __bfloat1622float2(pv[2]), x3 = __bfloat1622float2(pv[3]);
                    lam = fmaf(x0.x, l0.x, lam);
                    lam2 = fmaf(x0.y, l0.y, lam2);
                    lam = fmaf(x1.x, l0.z, lam);
                    lam2 = fmaf(x1.y, l0.w, lam2);
                    lam = fmaf(x2.x, l1.x, lam);
                    lam2 = fmaf(x2.y, l1.y, lam2);
                    lam = fmaf(x3.x, l1.z, lam);
                    lam2 = fmaf(x3.y, l1.w, lam2);
                }
            lam = (lam + lam2) * s.scale + sm.bias_c[cpar];
            gather_part(gth, 1);
            if (!mbar_wait(&sm.st_bar, st_phase)) {
                sm.abort_flag = 1;
                if (lane == 0) set_status(a.status, kDevTimeout);
            }
            tc_fence_after_sync();
            float sv[64], tv[64];
            tmem_ld64x2(t_lane, t_lane + 64, sv, tv);
            gather_part(gth, 2);
            // One exponential per key: e_j = exp(x_j - m) over the row's visible keys (x = scale s, four partial
            // maxima / sums so that no chain of 64 dependent operations forms); the final weights are e_j times one
            // factor per row: alpha / Z in a selected chunk, exp(m - lse) in the local span.
            const float c2 = s.scale * 1.4426950408889634f;         // scale * log2(e)
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int j = 0; j < 64; ++j) mx[j & 3] = fmaxf(mx[j & 3], j <= limit ? sv[j] : -INFINITY);
            float m = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
            if (limit < 0) m = 0.f;                                 // padding row
            const float m2 = m * c2;
            float Zp[4] = {0.f, 0.f, 0.f, 0.f}, gp[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int j = 0; j < 64; ++j) {
                float e;
                asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(fmaf(sv[j], c2, -m2)));
                e = j <= limit ? e : 0.f;
                sv[j] = e;
                Zp[j & 3] += e;
                gp[j & 3] = fmaf(e, tv[j], gp[j & 3]);
            }
            gather_part(gth, 3);
            const float Z = (Zp[0] + Zp[1]) + (Zp[2] + Zp[3]), gt = (gp[0] + gp[1]) + (gp[2] + gp[3]);
            m *= s.scale;
            float f, sub = dsum, dl = 0.f;
            if (!local) {
                const float gc = gt / Z;
                const float alpha = __expf(lam - lse);
                f = alpha / Z;
                sub = gc;
                dl = limit >= 0 ? alpha * (gc - dsum) * s.scale : 0.f;
            } else {
                f = __expf(m - lse);
            }
            if (limit < 0) {                                        // padding row: Z = 0, nothing may leak a NaN
                f = 0.f;
                sub = 0.f;
            }
            const float fs = f * s.scale;
#pragma unroll
            for (int j = 0; j < 64; ++j) {
                const float e = sv[j];
                sv[j] = e * fs * (tv[j] - sub);            // d s_j (times scale)
                tv[j] = e * f;                             // w_j
            }
#pragma unroll
            for (int pc = 0; pc < 8; ++pc) {
                *reinterpret_cast<uint4*>(dsbuf + swz128(row, pc)) =
                    make_uint4(pack_bf16(sv[8 * pc], sv[8 * pc + 1]), pack_bf16(sv[8 * pc + 2], sv[8 * pc + 3]),
                               pack_bf16(sv[8 * pc + 4], sv[8 * pc + 5]), pack_bf16(sv[8 * pc + 6], sv[8 * pc + 7]));
                *reinterpret_cast<uint4*>(wbuf + swz128(row, pc)) =
                    make_uint4(pack_bf16(tv[8 * pc], tv[8 * pc + 1]), pack_bf16(tv[8 * pc + 2], tv[8 * pc + 3]),
                               pack_bf16(tv[8 * pc + 4], tv[8 * pc + 5]), pack_bf16(tv[8 * pc + 6], tv[8 * pc + 7]));
            }
            sm.dlam[row] = dl;
            fence_proxy_async_smem();               // d S is an operand of the d Q MMA
            tc_fence_before_sync();
        }
        st_phase ^= 1u;
        if (has_next) store_row(nri, par ^ 1);
        asm volatile("cp.async.commit_group;" ::: "memory");
        if (has_next && !next_new) {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            fence_proxy_async_smem();
        }
        __syncthreads();                        // d S, W and d lambda of all 128 rows are in shared memory
        if (warp >= 4) {                        // what the deferred read-out of this tile needs
            const int row = (warp - 4) * 32 + lane;
            ro_orow = sm.row_orow[par][row];
            ro_dl = sm.dlam[row];
            ro_cpar = cpar;
        }
        ro_pending = true;
        if (tid == 0) {
            // d Q = d S K: A = d S as written above (K-major, 64 keys), B = the chunk's K tile read MN-major
            constexpr uint32_t idesc_dq = umma_idesc_bf16(kRows, kD) | kUmmaBMnMajor;
            tc_fence_after_sync();
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
                umma_bf16(tmem_base + 128, dds0 + ((ks * 32) >> 4), dkmn0 + ((ks * 2048) >> 4), idesc_dq, ks > 0 ? 1u : 0u);
            umma_commit(&sm.dq_bar);
            // dK^T += Q^T dS and dV^T += dO^T W: contractions over the tile's 128 rows; A = the Q / dO rows read MN-major
            // (dimension contiguous, the two 64-dim boxes 16 KB apart), B = d S / W read MN-major (key contiguous)
            constexpr uint32_t idesc_kv = umma_idesc_bf16(kD, kS) | kUmmaAMnMajor | kUmmaBMnMajor;
            const uint64_t dqmn0 = umma_desc_mn128(q_addr, kRows * 128, 1024u), ddmn0 = umma_desc_mn128(do_addr, kRows * 128, 1024u);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint32_t accf = (run_acc || ks > 0) ? 1u : 0u;
                umma_bf16(tmem_base + 256, dqmn0 + ((ks * 2048) >> 4), ddsmn0 + ((ks * 2048) >> 4), idesc_kv, accf);
                umma_bf16(tmem_base + 320, ddmn0 + ((ks * 2048) >> 4), dwmn0 + ((ks * 2048) >> 4), idesc_kv, accf);
            }
            umma_commit(&sm.p2_bar);
            // same chunk next: its S and T can start now (their operands are in place, S / T of this tile were read)
            if (has_next && !next_new)
                issue_st(smem_u32(qbuf0 + (par ^ 1) * kQBytes), smem_u32(dobuf0 + (par ^ 1) * kQBytes));
        }
        st_issued = has_next && !next_new;
        dq_phase ^= 1u;
        p2_phase ^= 1u;
        run_acc = true;

        // ------------------------------------------------------------------ d landmark, d bias (CUDA cores)
        if (warp >= 4) {
            // d landmark: sum over rows of (scale d lambda_r) q_r.  Warp w - 4 owns dims 32 (w - 4) .. +31 (one per
            // lane) and walks all 128 rows; the partial sums stay in a register until the chunk ends.
            const int dim = (warp - 4) * 32 + lane;
            const uint8_t* col = qbuf + (dim >> 6) * (kRows * 128) + (dim & 7) * 2;
            const int piece = (dim & 63) >> 3;
            float acc0 = 0.f, acc1 = 0.f;
#pragma unroll 8
            for (int r = 0; r < kRows; r += 2) {
                acc0 = fmaf(sm.dlam[r], __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(col + swz128(r, piece))), acc0);
                acc1 = fmaf(sm.dlam[r + 1], __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(col + swz128(r + 1, piece))), acc1);
            }
            lm_acc += acc0 + acc1;
            if (warp == 4) {
                const float v = sm.dlam[lane] + sm.dlam[lane + 32] + sm.dlam[lane + 64] + sm.dlam[lane + 96];
                bias_acc += warp_sum(v);
            }
        }
        // the next chunk's K, V and landmark may land once every MMA on this chunk has completed: its d Q is the last
        if (next_new && warp >= 4) {
            if (!mbar_wait(&sm.dq_bar, dq_phase ^ 1u)) {
                sm.abort_flag = 1;
                if (lane == 0) set_status(a.status, kDevTimeout);
            }
            issue_chunk(nrec.x, nrec.y, cpar ^ 1);
        }
        if (next_new) {
            kv_issued = true;
            cpar ^= 1;
        }
        if (!has_next || next_new) flush();
        rec = nrec;
        nrec = n2rec;
        nent = n2ent;
        n2rec = n3rec;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (warp >= 4 && ro_pending && !sm.abort_flag) read_out();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 0) tmem_dealloc(tmem_base, 512);
}

}  // namespace

bool prefill_backward_fast_supports(const Shape& s, int dtype) {
    return prefill_fast_supports(s, dtype) && s.Hl == s.Hkv && s.K + 17 <= 255 &&
           static_cast<long long>(s.B) * s.Hq * s.R < (1ll << 31);
}

namespace {
size_t dsum_bytes(const Shape& s) { return (static_cast<size_t>(s.B) * s.Hq * s.R * sizeof(float) + 255) / 256 * 256; }
}

size_t prefill_backward_fast_scratch_bytes(const Shape& s) { return dsum_bytes(s) + inverse_index_bytes(s); }

int launch_prefill_backward_fast(const Shape& s, const BackwardTensors& t, cudaStream_t stream) {
    if (t.scratch_bytes < prefill_backward_fast_scratch_bytes(s)) return HILS_ERR_WORKSPACE;
    char* sc = static_cast<char*>(t.scratch);
    float* dsum = reinterpret_cast<float*>(sc);
    const long long rows = static_cast<long long>(s.B) * s.Hq * s.R;
    int launches = 0;
    backward_dsum_kernel<<<static_cast<unsigned>((rows + 7) / 8), 256, 0, stream>>>(
        static_cast<const __nv_bfloat16*>(t.dout), static_cast<const __nv_bfloat16*>(t.out), dsum, rows);
    if (cudaGetLastError() != cudaSuccess) return HILS_ERR_CUDA;
    trace_mark("backward_dsum", stream);
    ++launches;

    InverseIndex ix;
    const int rc = build_inverse_index(s, t.sel_idx, sc + dsum_bytes(s), t.scratch_bytes - dsum_bytes(s), &ix, stream);
    if (rc < 0) return rc;
    launches += rc;

    CUtensorMap map_k, map_v;
    const uint64_t kv_rows = static_cast<uint64_t>(s.B) * s.Hkv * s.T;
    if (!make_bf16_2d_map(&map_k, t.k, kv_rows, kD, 64, kS) || !make_bf16_2d_map(&map_v, t.v, kv_rows, kD, 64, kS))
        return HILS_ERR_CUDA;
    const size_t smem = 2 * kKBytes + 4 * kQBytes + 2 * kDsBytes + sizeof(BtSmem) + 1024;
    // HILS_BACKWARD_MMA_SYNC=1: the warp-level variant (every product on mma.sync) instead of the tcgen05 one
    static const bool warp_mma = [] { const char* e = getenv("HILS_BACKWARD_MMA_SYNC"); return e && e[0] == '1'; }();
    static PerDeviceOnce attr_once;
    if (attr_once.pending()) {
        if (cudaFuncSetAttribute(prefill_backward_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem)) != cudaSuccess ||
            cudaFuncSetAttribute(prefill_backward_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem)) != cudaSuccess)
            return HILS_ERR_CUDA;
        attr_once.done();
    }
    BfArgs a;
    a.s = s;
    a.q = static_cast<const __nv_bfloat16*>(t.q);
    a.dout = static_cast<const __nv_bfloat16*>(t.dout);
    a.lm = static_cast<const __nv_bfloat16*>(t.landmarks);
    a.bias = t.bias;
    a.lse = t.lse;
    a.dsum = dsum;
    a.entries = ix.entries;
    a.tiles = ix.tiles;
    a.dq = t.dq;
    a.dk = t.dk;
    a.dv = t.dv;
    a.dlm = t.dlandmarks;
    a.dbias = t.dbias;
    a.status = t.status;
    for (int blk = 0; blk < ix.n_blocks; ++blk) {
        a.blk_range = ix.blk_toff + blk;
        a.i0 = blk * ix.qb;
        if (warp_mma) prefill_backward_mma_kernel<<<sm_count(), kBfThreads, smem, stream>>>(map_k, map_v, a);
        else prefill_backward_tc_kernel<<<sm_count(), kBfThreads, smem, stream>>>(map_k, map_v, a);
        if (cudaGetLastError() != cudaSuccess) return HILS_ERR_CUDA;
        trace_mark("backward_attend", stream);
        ++launches;
    }
    return launches;
}

}  // namespace hils
