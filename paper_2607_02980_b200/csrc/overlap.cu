// Chunk-id overlap among blocks of M adjacent queries (Sec. "Chunk Overlap", Eq. Overlap):
//     Overlap = (M K - |union_m I_m|) / ((M - 1) K),
// I_m the chunks retrieved by the m-th query of the block, plus the counts the section's figure is drawn from:
// the size of the union (what a packed kernel loads once per block) and how much of it the previous block had
// already loaded.  Integer work on the selection the operator wrote; nothing here is floating point except the
// final division.
//
// One warp walks a run of consecutive blocks of one (sequence, KV head) pair with two bit sets over the chunk
// ids in shared memory: `cur` collects the block's chunks with atomicOr (a chunk counts for the union when its
// bit was clear), `prev` holds the previous block's union for the reuse count.  After a block the older set is
// cleared by walking that block's ids again (a few words instead of the whole set) and the two swap roles.
// Warps are independent (no CTA-wide barrier); a CTA holds as many warps as its shared memory has room for sets.
#include "common.cuh"
#include "internal.h"

namespace hils {

namespace {

constexpr int kOvMaxWarps = 8;
constexpr size_t kOvSmemBudget = 64 * 1024;      // per CTA, unless a single warp's two sets need more

struct OvArgs {
    const int32_t* sel;     // [pairs, R, K]
    int32_t* stats;         // [pairs, nblk, 4]: total, union, reused, full
    float* overlap;         // [pairs, nblk] or null
    int pairs, R, K, C, M, nblk, blocks_per_run, runs_per_pair, words, vec4;
};

__global__ void __launch_bounds__(kOvMaxWarps * 32) chunk_overlap_kernel(const OvArgs a) {
    extern __shared__ unsigned ov_sets[];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5, wpc = blockDim.x >> 5;
    const long long run = static_cast<long long>(blockIdx.x) * wpc + wib;
    if (run >= static_cast<long long>(a.pairs) * a.runs_per_pair) return;
    const int pair = static_cast<int>(run / a.runs_per_pair);
    const int blk0 = static_cast<int>(run % a.runs_per_pair) * a.blocks_per_run;
    const int blk1 = min(a.nblk, blk0 + a.blocks_per_run);
    unsigned* cur = ov_sets + static_cast<size_t>(wib) * 2 * a.words;
    unsigned* prev = cur + a.words;

    for (int w = lane; w < 2 * a.words; w += 32) cur[w] = 0u;
    __syncwarp();
    const int32_t* psel = a.sel + static_cast<long long>(pair) * a.R * a.K;
    const int full_ent = a.M * a.K;
    // the block before this run's first one supplies the first `prev`
    if (blk0 > 0) {
        const int32_t* src = psel + static_cast<long long>(blk0 - 1) * full_ent;
#pragma unroll 4
        for (int e = lane; e < full_ent; e += 32) {
            const int id = __ldg(src + e);
            if (id >= 0 && id < a.C) atomicOr(&prev[id >> 5], 1u << (id & 31));
        }
        __syncwarp();
    }

    for (int blk = blk0; blk < blk1; ++blk) {
        const int nq = min(a.M, a.R - blk * a.M);
        const int nent = nq * a.K;
        const int32_t* src = psel + static_cast<long long>(blk) * full_ent;
        int tot = 0, uni = 0, reu = 0;
        auto visit = [&](int id) {
            if (id >= 0 && id < a.C) {
                ++tot;
                const unsigned bit = 1u << (id & 31);
                const unsigned old = atomicOr(&cur[id >> 5], bit);
                if (!(old & bit)) {
                    ++uni;
                    if (prev[id >> 5] & bit) ++reu;
                }
            }
        };
        if (a.vec4) {
            // K a multiple of 4 and a 16-byte aligned base: four ids per load, up to four loads in flight per lane
            const int4* src4 = reinterpret_cast<const int4*>(src);
#pragma unroll 4
            for (int e = lane; e < (nent >> 2); e += 32) {
                const int4 v = __ldg(src4 + e);
                visit(v.x);
                visit(v.y);
                visit(v.z);
                visit(v.w);
            }
        } else {
#pragma unroll 4
            for (int e = lane; e < nent; e += 32) visit(__ldg(src + e));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            tot += __shfl_xor_sync(kFullMask, tot, o);
            uni += __shfl_xor_sync(kFullMask, uni, o);
            reu += __shfl_xor_sync(kFullMask, reu, o);
        }
        if (lane == 0) {
            const bool full = nq == a.M && tot == full_ent;
            const long long o = static_cast<long long>(pair) * a.nblk + blk;
            reinterpret_cast<int4*>(a.stats)[o] = make_int4(tot, uni, reu, full ? 1 : 0);
            if (a.overlap)
                a.overlap[o] = full && a.M > 1
                                   ? static_cast<float>(full_ent - uni) / static_cast<float>((a.M - 1) * a.K)
                                   : __int_as_float(0x7fc00000);
        }
        // the older set becomes the next block's empty `cur`: clear the words of the block it was built from
        // (the shuffles above ordered every lane's reads of `prev` before these writes)
        if (blk > 0) {
            const int32_t* old_src = src - full_ent;
#pragma unroll 4
            for (int e = lane; e < full_ent; e += 32) {
                const int id = __ldg(old_src + e);
                if (id >= 0 && id < a.C) prev[id >> 5] = 0u;
            }
        }
        __syncwarp();
        unsigned* t = prev;
        prev = cur;
        cur = t;
    }
}

}  // namespace

bool chunk_overlap_supports(int C) { return C >= 1 && C <= (1 << 19); }

int launch_chunk_overlap(int pairs, int R, int K, int C, int M, const int32_t* sel, int32_t* stats, float* overlap,
                         cudaStream_t stream) {
    OvArgs a;
    a.sel = sel;
    a.stats = stats;
    a.overlap = overlap;
    a.pairs = pairs;
    a.R = R;
    a.K = K;
    a.C = C;
    a.M = M;
    a.nblk = (R + M - 1) / M;
    a.words = (C + 31) / 32;
    a.vec4 = (K % 4 == 0 && (reinterpret_cast<uintptr_t>(sel) & 15u) == 0) ? 1 : 0;
    const size_t per_warp = sizeof(unsigned) * 2 * a.words;
    int wpc = static_cast<int>(kOvSmemBudget / per_warp);
    wpc = wpc < 1 ? 1 : (wpc > kOvMaxWarps ? kOvMaxWarps : wpc);
    // enough runs for 32 warps per SM; a run never shorter than 8 blocks (each run re-reads one block to start)
    const int want_runs = (sm_count() * 32 + pairs - 1) / pairs;
    int per = (a.nblk + want_runs - 1) / want_runs;
    if (per < 8) per = 8;
    a.blocks_per_run = per;
    a.runs_per_pair = (a.nblk + per - 1) / per;
    const long long ctas = (static_cast<long long>(pairs) * a.runs_per_pair + wpc - 1) / wpc;
    if (ctas > 0x7fffffffll) return HILS_ERR_UNSUPPORTED;
    const size_t smem = per_warp * wpc;
    if (smem > 48 * 1024) {
        static PerDeviceOnce attr_once;
        if (attr_once.pending()) {
            if (cudaFuncSetAttribute(chunk_overlap_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 1024) !=
                cudaSuccess)
                return HILS_ERR_CUDA;
            attr_once.done();
        }
    }
    chunk_overlap_kernel<<<static_cast<unsigned>(ctas), wpc * 32, smem, stream>>>(a);
    if (cudaGetLastError() != cudaSuccess) return HILS_ERR_CUDA;
    return 1;
}

}  // namespace hils
