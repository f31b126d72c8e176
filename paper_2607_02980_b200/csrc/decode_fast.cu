// Bandwidth-tuned decode kernels: bf16, d = 128, S = 64, G <= 8, one landmark per KV head, W = 1.
//
//   decode_score   streams the landmarks of every (sequence, KV head) once with 128-bit loads and
//                  scores them against the G query heads with warp MMA (landmark rows are the A
//                  operand straight from global memory); writes the group score u_c = max_h s^h_c.
//   decode_select  one CTA per (sequence, KV head): exact top-K of u (ties to the lower chunk id),
//                  ascending ids, then the per-head surrogate scores of the selected chunks and the
//                  fusion weights exp(s^h_c - max_c s^h_c).
//   decode_attend  persistent CTAs over a flat list of (pair, slot) items; K/V chunks arrive through
//                  a TMA + mbarrier ring (128B-swizzled tiles), each consumer warp runs one chunk at
//                  a time: QK^T, the chunk's own softmax, PV (Eq. HiLS weights); the CTA that
//                  finishes a pair last mixes the partial sums with the local branch (App. C).
#include "internal.h"
#include "tma.cuh"

namespace hils {
namespace {

constexpr int kD = 128;
constexpr int kS = 64;
constexpr int kScoreThreads = 256;
constexpr int kScoreChunksPerCta = 256;      // 8 warps x 2 iterations x 16 chunks
constexpr int kSelThreads = 512;
constexpr int kSelBins = 2048;
constexpr int kSelCap = 1024;                // candidates ranked exactly in shared memory
constexpr int kStages = 5;
constexpr int kStageBytes = 2 * kS * kD * 2; // K tile + V tile
constexpr int kMaxItems = 2048;
constexpr int kConsumerWarps = 5;       // == kStages: a stage is always consumed by the same warp, so no
                                        // waiter can ever be more than one mbarrier phase away from its stage
static_assert(kStages % kConsumerWarps == 0, "stage ownership must be fixed per consumer warp");
constexpr int kAttendThreads = (kConsumerWarps + 1) * 32;
constexpr float kLog2e = 1.4426950408889634f;

struct DArgs {
    Shape s;
    const __nv_bfloat16* q;
    const __nv_bfloat16* lm;
    const float* bias;
    const int32_t* seq_lens;
    __nv_bfloat16* out;
    float* lse;
    int32_t* sel;
    int* status;
    // scratch
    float* u;          // [pairs, Cpad] group scores
    int Cpad;
    float* wgt;        // [pairs, G, K] exp(s^h_c - R_h) of the selected chunks
    float* Rh;         // [pairs, G]    max_c s^h_c over the selected chunks
    float* Eh;         // [pairs, G]    sum of wgt
    int* pair_n;       // [pairs]       number of selected chunks, -1 = invalid sequence length
    int* done;         // [pairs]       slots finished (zeroed by the selection)
    float* part;       // [pairs, max_parts, G, 128] weighted partial sums
    float* loc_o;      // [pairs, G, 128] local-branch output
    float* loc_lam;    // [pairs, G]      log Z_swa
    int max_parts;
    int n_ctas;
};

// ------------------------------------------------------------------------------------------ select
__device__ inline int block_excl_scan(int v, int* warp_tot, int& total) {
    // exclusive prefix of v over the block in thread order; warp_tot: shared int[32]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(kFullMask, inc, o);
        if (lane >= o) inc += n;
    }
    __syncthreads();
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    int base = 0, tot = 0;
    for (int w = 0; w < nw; ++w) {
        const int x = warp_tot[w];
        if (w < warp) base += x;
        tot += x;
    }
    total = tot;
    return base + inc - v;
}

struct SelShared {
    int hist[kSelBins];
    unsigned long long cand[kSelCap];
    int sel_s[128];
    float lam_s[8][128];
    alignas(16) __nv_bfloat16 lm_s[64][kD + 8];    // selected landmark rows, 64 at a time (padded rows)
    alignas(16) __nv_bfloat16 q_s[8][kD + 8];
    int warp_tot[32];
    int sh_i[8];
    int is_last;
};

// Exact top-K of the group scores of one (sequence, KV head) pair (ties: lower chunk id), ascending ids,
// then the per-head surrogate scores of the selected chunks and the fusion weights.  Called by every
// thread of the CTA that finished the pair's scoring last; u was written by other CTAs (L2 reads).
__device__ void select_pair(const DArgs& a, int pair, int ncand, SelShared& sh) {
    const Shape& s = a.s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, NT = blockDim.x;
    const int b = pair / s.Hkv, g = pair % s.Hkv;
    const int K = s.K, G = s.G;
    int32_t* sel = a.sel + static_cast<long long>(pair) * K;
    const int n = min(K, ncand);
    const float* u = a.u + static_cast<long long>(pair) * a.Cpad;
    int* hist = sh.hist;
    int* sel_s = sh.sel_s;
    int* sh_i = sh.sh_i;

    if (ncand <= K) {
        for (int t = tid; t < K; t += NT) sel_s[t] = t < ncand ? t : -1;
        __syncthreads();
    } else if (ncand <= 8 * NT) {
        // --- short candidate lists: every thread keeps 8 consecutive ordered keys in registers and the
        //     K-th best is found with a 4 x 8-bit radix select (shared-memory histograms only)
        unsigned key[8];
        const int cb = tid * 8;
#pragma unroll
        for (int i = 0; i < 8; ++i) key[i] = cb + i < ncand ? ordered_key(__ldcg(u + cb + i)) : 0u;
        unsigned prefix = 0u;
        int remaining = K, n_eq = 0;
#pragma unroll 1
        for (int shift = 24; shift >= 0; shift -= 8) {
            if (tid < 256) hist[tid] = 0;
            __syncthreads();
            const unsigned himask = shift == 24 ? 0u : (0xffffffffu << (shift + 8));
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (cb + i < ncand && (key[i] & himask) == (prefix & himask)) atomicAdd(&hist[(key[i] >> shift) & 255u], 1);
            __syncthreads();
            if (warp == 0) {
                // lane l owns digits 255-8l .. 248-8l (top-down)
                int loc[8], tsum = 0;
#pragma unroll
                for (int x = 0; x < 8; ++x) { loc[x] = hist[255 - 8 * lane - x]; tsum += loc[x]; }
                int inc = tsum;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int nn = __shfl_up_sync(kFullMask, inc, o);
                    if (lane >= o) inc += nn;
                }
                int cum = inc - tsum;
                if (cum < remaining && inc >= remaining) {
#pragma unroll
                    for (int x = 0; x < 8; ++x) {
                        if (cum + loc[x] >= remaining) { sh_i[4] = 255 - 8 * lane - x; sh_i[5] = cum; sh_i[6] = loc[x]; break; }
                        cum += loc[x];
                    }
                }
            }
            __syncthreads();
            prefix |= static_cast<unsigned>(sh_i[4]) << shift;
            remaining -= sh_i[5];
            n_eq = sh_i[6];
        }
        // prefix = key of the K-th best; `remaining` of the n_eq chunks with that key are taken, lowest ids first
        int eq_before = 0, tot;
        if (n_eq != remaining) {                        // ties across the cut (block-uniform branch)
            int eq = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) eq += (cb + i < ncand && key[i] == prefix) ? 1 : 0;
            eq_before = block_excl_scan(eq, sh.warp_tot, tot);
        }
        int cnt = 0, e = eq_before;
        unsigned take = 0u;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (cb + i >= ncand) continue;
            bool tk = key[i] > prefix;
            if (key[i] == prefix) { tk = n_eq == remaining || e < remaining; ++e; }
            if (tk) { take |= 1u << i; ++cnt; }
        }
        int pos = block_excl_scan(cnt, sh.warp_tot, tot);
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (take & (1u << i)) sel_s[pos++] = cb + i;
        __syncthreads();
    } else {
        // --- 1. value range
        float mn = INFINITY, mx = -INFINITY;
        for (int c = tid; c < ncand; c += NT) { const float v = __ldcg(u + c) + 0.f; mn = fminf(mn, v); mx = fmaxf(mx, v); }
        mn = -warp_max(-mn); mx = warp_max(mx);
        if (lane == 0) { sh.lam_s[0][warp] = mn; sh.lam_s[1][warp] = mx; }
        for (int i = tid; i < kSelBins; i += NT) hist[i] = 0;
        if (tid == 0) sh_i[3] = 0;
        __syncthreads();
        float lo = sh.lam_s[0][0], hi = sh.lam_s[1][0];
        for (int w = 1; w < NT / 32; ++w) { lo = fminf(lo, sh.lam_s[0][w]); hi = fmaxf(hi, sh.lam_s[1][w]); }
        const float inv = (hi > lo) ? static_cast<float>(kSelBins - 1) / (hi - lo) : 0.f;
        __syncthreads();
        // --- 2. histogram over a monotone linear binning
        for (int c = tid; c < ncand; c += NT) {
            const int bin = max(0, min(kSelBins - 1, static_cast<int>((__ldcg(u + c) + 0.f - lo) * inv)));
            atomicAdd(&hist[bin], 1);
        }
        __syncthreads();
        // --- 3. boundary bin: the highest bin b* with count(bin >= b*) >= K.  Thread i owns the
        //        kSelBins / NT bins below (kSelBins - 1 - i * per); a block scan gives the count above.
        {
            const int per = kSelBins / NT;
            const int top = kSelBins - 1 - tid * per;
            int tsum = 0;
            for (int x = 0; x < per; ++x) tsum += hist[top - x];
            int tot;
            int cum = block_excl_scan(tsum, sh.warp_tot, tot);
            if (cum < K && cum + tsum >= K) {
                for (int x = 0; x < per; ++x) {
                    const int hb = hist[top - x];
                    if (cum + hb >= K) { sh_i[0] = top - x; sh_i[1] = cum + hb; sh_i[2] = cum; break; }
                    cum += hb;
                }
            }
        }
        __syncthreads();
        const int bstar = sh_i[0], m_cand = sh_i[1];
        if (m_cand <= kSelCap) {
            // --- 4a. gather the candidates and rank them exactly (score desc, id asc)
            unsigned long long* cand = sh.cand;
            for (int c = tid; c < ncand; c += NT) {
                const float v = __ldcg(u + c);
                const int bin = max(0, min(kSelBins - 1, static_cast<int>((v + 0.f - lo) * inv)));
                if (bin >= bstar) cand[atomicAdd(&sh_i[3], 1)] = select_key(v, c);
            }
            __syncthreads();
            unsigned long long mine[kSelCap / kSelThreads];
            bool keep[kSelCap / kSelThreads];
#pragma unroll
            for (int r = 0; r < kSelCap / kSelThreads; ++r) {
                const int i = tid + r * NT;
                mine[r] = i < m_cand ? cand[i] : 0ull;
                int rank = 0;
                if (i < m_cand)
                    for (int j = 0; j < m_cand; ++j) rank += cand[j] > mine[r] ? 1 : 0;
                keep[r] = i < m_cand && rank < K;                  // ranks are unique
            }
            __syncthreads();
#pragma unroll
            for (int r = 0; r < kSelCap / kSelThreads; ++r) {
                const int i = tid + r * NT;
                if (i < m_cand && !keep[r]) cand[i] = 0ull;
            }
            __syncthreads();
            // ascending ids: position = number of selected ids below mine
#pragma unroll
            for (int r = 0; r < kSelCap / kSelThreads; ++r) {
                if (!keep[r]) continue;
                const int id = key_chunk(mine[r]);
                int pos = 0;
                for (int j = 0; j < m_cand; ++j) {
                    const unsigned long long o = cand[j];
                    pos += (o != 0ull && key_chunk(o) < id) ? 1 : 0;
                }
                sel_s[pos] = id;
            }
            __syncthreads();
        } else {
            // --- 4b. many equal / clustered scores: exact 4 x 8-bit radix select on the ordered key,
            //         then an ordered scan (each thread owns a contiguous range of chunk ids)
            unsigned prefix = 0u;
            int remaining = K;
            for (int shift = 24; shift >= 0; shift -= 8) {
                for (int i = tid; i < 256; i += NT) hist[i] = 0;
                __syncthreads();
                const unsigned himask = shift == 24 ? 0u : (0xffffffffu << (shift + 8));
                for (int c = tid; c < ncand; c += NT) {
                    const unsigned key = ordered_key(__ldcg(u + c));
                    if ((key & himask) == (prefix & himask)) atomicAdd(&hist[(key >> shift) & 255u], 1);
                }
                __syncthreads();
                if (tid == 0) {
                    int cum = 0, dsel = 0;
                    for (int dgt = 255; dgt >= 0; --dgt) {
                        if (cum + hist[dgt] >= remaining) { dsel = dgt; break; }
                        cum += hist[dgt];
                    }
                    sh_i[4] = dsel; sh_i[5] = cum;
                }
                __syncthreads();
                prefix |= static_cast<unsigned>(sh_i[4]) << shift;
                remaining -= sh_i[5];
                __syncthreads();
            }
            // prefix = key of the K-th best; `remaining` of the chunks with that key are taken, lowest ids first
            const int per = (ncand + NT - 1) / NT;
            const int cb = min(ncand, tid * per), ce = min(ncand, cb + per);
            int eq = 0;
            for (int c = cb; c < ce; ++c) eq += ordered_key(__ldcg(u + c)) == prefix ? 1 : 0;
            int tot;
            int eq_before = block_excl_scan(eq, sh.warp_tot, tot);
            int cnt = 0;
            int e = eq_before;
            for (int c = cb; c < ce; ++c) {
                const unsigned key = ordered_key(__ldcg(u + c));
                if (key > prefix) ++cnt;
                else if (key == prefix) { if (e < remaining) ++cnt; ++e; }
            }
            int pos = block_excl_scan(cnt, sh.warp_tot, tot);
            e = eq_before;
            for (int c = cb; c < ce; ++c) {
                const unsigned key = ordered_key(__ldcg(u + c));
                bool take = key > prefix;
                if (key == prefix) { take = e < remaining; ++e; }
                if (take) sel_s[pos++] = c;
            }
            __syncthreads();
        }
    }
    for (int t = tid; t < K; t += NT) sel[t] = t < n ? sel_s[t] : -1;

    // --- 5. per-head surrogate scores of the selected chunks and the fusion weights: the selected
    //        landmark rows and the G queries are staged in shared memory with one round of 16-byte
    //        loads, then every thread computes one (chunk, head) dot product
    const __nv_bfloat16* lm = a.lm + static_cast<long long>(pair) * s.C * kD;
    const __nv_bfloat16* qg = a.q + (static_cast<long long>(b) * s.Hq + g * G) * kD;
    for (int x = tid; x < G * 16; x += NT)
        *reinterpret_cast<uint4*>(&sh.q_s[x >> 4][(x & 15) * 8]) = *reinterpret_cast<const uint4*>(qg + (x >> 4) * kD + (x & 15) * 8);
    for (int t0 = 0; t0 < n; t0 += 64) {
        const int nt = min(64, n - t0);
        __syncthreads();
        for (int x = tid; x < nt * 16; x += NT) {
            const int t = x >> 4, pc = x & 15;
            *reinterpret_cast<uint4*>(&sh.lm_s[t][pc * 8]) =
                *reinterpret_cast<const uint4*>(lm + static_cast<long long>(sel_s[t0 + t]) * kD + pc * 8);
        }
        __syncthreads();
        for (int x = tid; x < nt * G; x += NT) {
            const int t = x / G, h = x % G;
            const __nv_bfloat16* lr = sh.lm_s[t];
            const __nv_bfloat16* qr = sh.q_s[h];
            float acc = 0.f;
#pragma unroll 8
            for (int e = 0; e < kD; e += 2) {
                const float2 lv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(lr + e));
                const float2 qv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(qr + e));
                acc = fmaf(lv.x, qv.x, acc);
                acc = fmaf(lv.y, qv.y, acc);
            }
            const float bb = a.bias ? a.bias[static_cast<long long>(pair) * s.C + sel_s[t0 + t]] : 0.f;
            sh.lam_s[h][t0 + t] = acc * s.scale + bb;
        }
    }
    __syncthreads();
    if (warp < G) {
        const int h = warp;
        float mx = -INFINITY;
        for (int t = lane; t < n; t += 32) mx = fmaxf(mx, sh.lam_s[h][t]);
        mx = warp_max(mx);
        float sum = 0.f;
        float* w = a.wgt + (static_cast<long long>(pair) * G + h) * K;
        for (int t = lane; t < K; t += 32) {
            const float e = t < n ? __expf(sh.lam_s[h][t] - mx) : 0.f;
            w[t] = e;
            sum += e;
        }
        sum = warp_sum(sum);
        if (lane == 0) { a.Rh[pair * G + h] = mx; a.Eh[pair * G + h] = sum; }
    }
    if (tid == 0) { a.pair_n[pair] = n; a.done[pair] = 0; }
}

// ------------------------------------------------------------------------------------------ score
__global__ void __launch_bounds__(kScoreThreads) decode_score_kernel(const DArgs a) {
    const Shape& s = a.s;
    const int pair = blockIdx.y;
    const int b = pair / s.Hkv, g = pair % s.Hkv;
    const int seq = a.seq_lens[b];
    if (seq < 1 || seq > s.T) return;
    const int ncand = (seq - 1) / kS;
    const int c_begin = blockIdx.x * kScoreChunksPerCta;
    if (c_begin >= ncand) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gq = lane >> 2, t = lane & 3;

    // B operand: q^T with the k index permuted so that each thread's 8 consecutive elements of a
    // 32-wide block feed two MMAs (the same permutation is applied to the landmark rows).
    uint4 qf[4];
#pragma unroll
    for (int kb = 0; kb < 4; ++kb) qf[kb] = make_uint4(0u, 0u, 0u, 0u);
    if (gq < s.G) {
        const __nv_bfloat16* qrow = a.q + (static_cast<long long>(b) * s.Hq + g * s.G + gq) * kD;
#pragma unroll
        for (int kb = 0; kb < 4; ++kb) qf[kb] = *reinterpret_cast<const uint4*>(qrow + kb * 32 + t * 8);
    }
    const __nv_bfloat16* lm = a.lm + static_cast<long long>(pair) * s.C * kD;
    const float* bias = a.bias ? a.bias + static_cast<long long>(pair) * s.C : nullptr;
    float* u = a.u + static_cast<long long>(pair) * a.Cpad;

    uint4 x[2][2][4];
    int c0[2];
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        c0[it] = c_begin + (warp * 2 + it) * 16;
        if (c0[it] < ncand) {
            const int r0 = min(c0[it] + gq, ncand - 1), r1 = min(c0[it] + gq + 8, ncand - 1);
#pragma unroll
            for (int kb = 0; kb < 4; ++kb) {
                x[it][0][kb] = __ldg(reinterpret_cast<const uint4*>(lm + static_cast<long long>(r0) * kD + kb * 32 + t * 8));
                x[it][1][kb] = __ldg(reinterpret_cast<const uint4*>(lm + static_cast<long long>(r1) * kD + kb * 32 + t * 8));
            }
        }
    }
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        if (c0[it] >= ncand) continue;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int kb = 0; kb < 4; ++kb) {
            const uint32_t a1[4] = {x[it][0][kb].x, x[it][1][kb].x, x[it][0][kb].y, x[it][1][kb].y};
            mma_bf16_16816(acc, a1, qf[kb].x, qf[kb].y);
            const uint32_t a2[4] = {x[it][0][kb].z, x[it][1][kb].z, x[it][0][kb].w, x[it][1][kb].w};
            mma_bf16_16816(acc, a2, qf[kb].z, qf[kb].w);
        }
        // acc[0..1]: chunk c0+gq, heads 2t, 2t+1; acc[2..3]: chunk c0+gq+8
        const bool h0 = 2 * t < s.G, h1 = 2 * t + 1 < s.G;
        float m0 = fmaxf(h0 ? acc[0] : -INFINITY, h1 ? acc[1] : -INFINITY);
        float m1 = fmaxf(h0 ? acc[2] : -INFINITY, h1 ? acc[3] : -INFINITY);
        m0 = fmaxf(m0, __shfl_xor_sync(kFullMask, m0, 1));
        m1 = fmaxf(m1, __shfl_xor_sync(kFullMask, m1, 1));
        m0 = fmaxf(m0, __shfl_xor_sync(kFullMask, m0, 2));
        m1 = fmaxf(m1, __shfl_xor_sync(kFullMask, m1, 2));
        const int ca = c0[it] + gq, cb = ca + 8;
        if (t == 0 && ca < ncand) u[ca] = m0 * s.scale + (bias ? bias[ca] : 0.f);
        if (t == 1 && cb < ncand) u[cb] = m1 * s.scale + (bias ? bias[cb] : 0.f);
    }
    pdl_launch_dependents();
}

// One CTA per (sequence, KV head) pair.
__global__ void __launch_bounds__(kSelThreads) decode_select_kernel(const DArgs a) {
    __shared__ SelShared sh;
    const Shape& s = a.s;
    const int pair = blockIdx.x, tid = threadIdx.x;
    const int b = pair / s.Hkv, g = pair % s.Hkv;
    const int seq = a.seq_lens[b];
    if (seq < 1 || seq > s.T) {
        // invalid length: flag it, emit empty outputs
        if (tid == 0) { set_status(a.status, kDevBadIndex); a.pair_n[pair] = -1; a.done[pair] = 0; }
        for (int t = tid; t < s.K; t += kSelThreads) a.sel[static_cast<long long>(pair) * s.K + t] = -1;
        for (int x = tid; x < s.G * kD; x += kSelThreads)
            a.out[(static_cast<long long>(b) * s.Hq + g * s.G) * kD + x] = __float2bfloat16_rn(0.f);
        if (tid < s.G) a.lse[static_cast<long long>(b) * s.Hq + g * s.G + tid] = 0.f;
        return;
    }
    pdl_wait();                                        // group scores of decode_score are visible
    select_pair(a, pair, (seq - 1) / kS, sh);
    pdl_launch_dependents();
}

// ------------------------------------------------------------------------------------------ attend
struct AttendSmem {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    int item_chunk[kMaxItems];     // chunk id, or -1 for an empty slot
    int item_nvalid[kMaxItems];    // valid rows (64, or fewer for the partial local chunk)
    float red[kConsumerWarps][8 * kD];
    int flag;
    int dead;                      // a bounded wait ran out: every consumer warp leaves at the next barrier
};

// first CTA whose item range [cta*N/n_ctas, (cta+1)*N/n_ctas) holds item x
__device__ inline int cta_of_item(long long x, long long N, int n_ctas) {
    return static_cast<int>(((x + 1) * n_ctas + N - 1) / N - 1);
}

// S = Q K^T for one 64-key tile held in shared memory (two 128B-swizzled boxes of 64 dims).
__device__ inline void qk_tile(const uint32_t (&aq)[8][2], uint32_t ks_addr, int lane, float (&sc)[8][4]) {
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
            const uint32_t a0[4] = {aq[2 * kp][0], 0u, aq[2 * kp][1], 0u};
            mma_bf16_16816(sc[nt], a0, r0, r1);
            const uint32_t a1[4] = {aq[2 * kp + 1][0], 0u, aq[2 * kp + 1][1], 0u};
            mma_bf16_16816(sc[nt], a1, r2, r3);
        }
    }
}

// O += P V for one 64-key tile; p holds the (already weighted) probabilities of rows g in [0], [1].
__device__ inline void pv_tile(const float (&p)[8][4], uint32_t vs_addr, int lane, float (&o)[16][4]) {
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
        const uint32_t ap[4] = {pack_bf16(p[2 * kk][0], p[2 * kk][1]), 0u, pack_bf16(p[2 * kk + 1][0], p[2 * kk + 1][1]), 0u};
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

__global__ void __launch_bounds__(kAttendThreads, 1)
decode_attend_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                     const DArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    AttendSmem& sm = *reinterpret_cast<AttendSmem*>(ring + kStages * kStageBytes);
    const Shape& s = a.s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int K = s.K, G = s.G, slots = K + 1;
    const long long N = static_cast<long long>(s.B) * s.Hkv * slots;
    const long long lo = (static_cast<long long>(blockIdx.x) * N) / a.n_ctas;
    const long long hi = (static_cast<long long>(blockIdx.x + 1) * N) / a.n_ctas;
    const int nitems = static_cast<int>(hi - lo);

    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], 1); }
        mbar_fence_init();
        sm.dead = 0;
        tma_prefetch_desc(&map_k);
        tma_prefetch_desc(&map_v);
    }
    pdl_wait();                                   // selection, weights and counters are visible
    for (int j = tid; j < nitems; j += kAttendThreads) {
        const long long idx = lo + j;
        const int pair = static_cast<int>(idx / slots), slot = static_cast<int>(idx % slots);
        const int n = a.pair_n[pair];
        int c = -1, nv = kS;
        if (n >= 0) {
            if (slot < K) {
                c = slot < n ? a.sel[static_cast<long long>(pair) * K + slot] : -1;
            } else {
                const int seq = a.seq_lens[pair / s.Hkv];
                c = (seq - 1) / kS;
                nv = (seq - 1) % kS + 1;
            }
        }
        sm.item_chunk[j] = c;
        sm.item_nvalid[j] = nv;
    }
    __syncthreads();
    if (nitems == 0) return;

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------------ producer (one lane)
        if (lane == 0) {
            for (int j = 0; j < nitems; ++j) {
                const int st = j % kStages;
                if (j >= kStages && !mbar_wait(&sm.empty[st], ((j / kStages) - 1) & 1)) {
                    set_status(a.status, kDevTimeout);
                    break;
                }
                const int c = sm.item_chunk[j];
                if (c < 0) { mbar_arrive(&sm.full[st]); continue; }
                const int pair = static_cast<int>((lo + j) / slots);
                const int row = pair * s.T + c * kS;
                uint8_t* dst = ring + st * kStageBytes;
                mbar_expect_tx(&sm.full[st], kStageBytes);
                tma_load_2d(dst, &map_k, &sm.full[st], 0, row);
                tma_load_2d(dst + 8192, &map_k, &sm.full[st], 64, row);
                tma_load_2d(dst + 16384, &map_v, &sm.full[st], 0, row);
                tma_load_2d(dst + 24576, &map_v, &sm.full[st], 64, row);
            }
        }
        return;
    }

    // ---------------------------------------------------------------------- consumers (5 warps)
    const int gq = lane >> 2, t = lane & 3;
    const float sl2 = s.scale * kLog2e;
    bool dead = false;
    int j0 = 0;
    while (j0 < nitems) {
        const int pair = static_cast<int>((lo + j0) / slots);
        const long long pair_end = static_cast<long long>(pair + 1) * slots;
        const int j1 = static_cast<int>(min(static_cast<long long>(nitems), pair_end - lo));
        const int b = pair / s.Hkv, g = pair % s.Hkv;
        const int n_sel = a.pair_n[pair];

        // A operand: the G query heads of this pair in rows 0..G-1
        uint32_t aq[8][2];
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) { aq[ks][0] = 0u; aq[ks][1] = 0u; }
        if (gq < G) {
            const __nv_bfloat16* qrow = a.q + (static_cast<long long>(b) * s.Hq + g * G + gq) * kD;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                aq[ks][0] = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 2 * t);
                aq[ks][1] = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8 + 2 * t);
            }
        }
        float o[16][4];
#pragma unroll
        for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;

        for (int j = j0 + ((warp - j0 % kConsumerWarps + kConsumerWarps) % kConsumerWarps); j < j1 && !dead;
             j += kConsumerWarps) {
            const int st = j % kStages;
            if (!mbar_wait(&sm.full[st], (j / kStages) & 1)) {
                if (lane == 0) { set_status(a.status, kDevTimeout); atomicExch(&sm.dead, 1); }
                dead = true;
                break;
            }
            const int c = sm.item_chunk[j];
            if (c >= 0) {
                const int slot = static_cast<int>((lo + j) % slots);
                const uint32_t ks_addr = smem_u32(ring + st * kStageBytes);
                const uint32_t vs_addr = ks_addr + 16384;
                float sc[8][4];
                qk_tile(aq, ks_addr, lane, sc);
                if (slot < K) {
                    // selected chunk: its own softmax, weighted by exp(s^h_c - R_h)
                    float m = -INFINITY;
#pragma unroll
                    for (int nt = 0; nt < 8; ++nt) m = fmaxf(m, fmaxf(sc[nt][0], sc[nt][1]));
                    m = fmaxf(m, __shfl_xor_sync(kFullMask, m, 1));
                    m = fmaxf(m, __shfl_xor_sync(kFullMask, m, 2));
                    float z = 0.f;
#pragma unroll
                    for (int nt = 0; nt < 8; ++nt) {
                        sc[nt][0] = exp2f((sc[nt][0] - m) * sl2);
                        sc[nt][1] = exp2f((sc[nt][1] - m) * sl2);
                        z += sc[nt][0] + sc[nt][1];
                    }
                    z += __shfl_xor_sync(kFullMask, z, 1);
                    z += __shfl_xor_sync(kFullMask, z, 2);
                    const float w = gq < G ? a.wgt[(static_cast<long long>(pair) * G + gq) * K + slot] / z : 0.f;
#pragma unroll
                    for (int nt = 0; nt < 8; ++nt) { sc[nt][0] *= w; sc[nt][1] *= w; }
                    pv_tile(sc, vs_addr, lane, o);
                } else {
                    // local branch: causal within the query's own (possibly partial) chunk
                    const int nv = sm.item_nvalid[j];
                    if (nv < kS) {
                        // rows past the sequence end may hold anything: zero them before P V
                        uint8_t* vt = ring + st * kStageBytes + 16384;
                        for (int x = lane; x < (kS - nv) * 16; x += 32) {
                            const int row = nv + (x >> 4), piece = x & 15;
                            *reinterpret_cast<uint4*>(vt + (piece >> 3) * 8192 + swz128(row, piece & 7)) =
                                make_uint4(0u, 0u, 0u, 0u);
                        }
                        __syncwarp();
                    }
                    float m = -INFINITY;
#pragma unroll
                    for (int nt = 0; nt < 8; ++nt) {
                        const int key = nt * 8 + 2 * t;
                        if (key >= nv) sc[nt][0] = -INFINITY;
                        if (key + 1 >= nv) sc[nt][1] = -INFINITY;
                        m = fmaxf(m, fmaxf(sc[nt][0], sc[nt][1]));
                    }
                    m = fmaxf(m, __shfl_xor_sync(kFullMask, m, 1));
                    m = fmaxf(m, __shfl_xor_sync(kFullMask, m, 2));
                    float z = 0.f;
#pragma unroll
                    for (int nt = 0; nt < 8; ++nt) {
                        sc[nt][0] = exp2f((sc[nt][0] - m) * sl2);
                        sc[nt][1] = exp2f((sc[nt][1] - m) * sl2);
                        z += sc[nt][0] + sc[nt][1];
                    }
                    z += __shfl_xor_sync(kFullMask, z, 1);
                    z += __shfl_xor_sync(kFullMask, z, 2);
                    const float w = 1.f / z;
#pragma unroll
                    for (int nt = 0; nt < 8; ++nt) { sc[nt][0] *= w; sc[nt][1] *= w; }
                    float ol[16][4];
#pragma unroll
                    for (int i = 0; i < 16; ++i) ol[i][0] = ol[i][1] = ol[i][2] = ol[i][3] = 0.f;
                    pv_tile(sc, vs_addr, lane, ol);
                    if (gq < G) {
                        float* dst = a.loc_o + (static_cast<long long>(pair) * G + gq) * kD;
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            *reinterpret_cast<float2*>(dst + i * 8 + 2 * t) = make_float2(ol[i][0], ol[i][1]);
                        if (t == 0) a.loc_lam[pair * G + gq] = m * s.scale + __logf(z);
                    }
                    if (nv < kS) fence_proxy_async_smem();
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.empty[st]);
        }

        // ---- end of this pair's items in this CTA: reduce the consumer warps, publish the partial sum
        if (gq < G) {
#pragma unroll
            for (int i = 0; i < 16; ++i)
                *reinterpret_cast<float2*>(&sm.red[warp][gq * kD + i * 8 + 2 * t]) = make_float2(o[i][0], o[i][1]);
        }
        asm volatile("bar.sync 1, %0;" ::"r"(kConsumerWarps * 32));
        dead = *reinterpret_cast<volatile int*>(&sm.dead) != 0;     // same value in all consumer threads
        const int first_cta = cta_of_item(static_cast<long long>(pair) * slots, N, a.n_ctas);
        const int part_idx = static_cast<int>(blockIdx.x) - first_cta;
        if (n_sel >= 0 && part_idx < a.max_parts) {
            float* dst = a.part + (static_cast<long long>(pair) * a.max_parts + part_idx) * G * kD;
            for (int x = tid; x < G * kD; x += kConsumerWarps * 32)
                dst[x] = ((sm.red[0][x] + sm.red[1][x]) + (sm.red[2][x] + sm.red[3][x])) + sm.red[4][x];
        }
        __threadfence();
        asm volatile("bar.sync 1, %0;" ::"r"(kConsumerWarps * 32));
        if (tid == 0) {
            const int covered = j1 - j0;
            const int old = atomicAdd(&a.done[pair], covered);
            sm.flag = (old + covered == slots) ? 1 : 0;
        }
        asm volatile("bar.sync 1, %0;" ::"r"(kConsumerWarps * 32));
        if (sm.flag && n_sel >= 0 && !dead) {
            // ---- last CTA of this pair: mix selected chunks and local branch (Eq. HiLS weights)
            __threadfence();
            const int last_cta = cta_of_item(pair_end - 1, N, a.n_ctas);
            const int nparts = min(a.max_parts, last_cta - first_cta + 1);
            for (int x = tid; x < G * kD; x += kConsumerWarps * 32) {
                const int h = x / kD;
                float A = 0.f;
                const float* src = a.part + static_cast<long long>(pair) * a.max_parts * G * kD + x;
                for (int pidx = 0; pidx < nparts; ++pidx) A += __ldcg(src + static_cast<long long>(pidx) * G * kD);
                const float lam_loc = __ldcg(a.loc_lam + pair * G + h);
                const float ol = __ldcg(a.loc_o + static_cast<long long>(pair) * G * kD + x);
                float res, lse;
                if (n_sel == 0) {
                    res = ol;
                    lse = lam_loc;
                } else {
                    const float R = a.Rh[pair * G + h], E = a.Eh[pair * G + h];
                    const float Rp = fmaxf(lam_loc, R);
                    const float wl = __expf(lam_loc - Rp), ws = __expf(R - Rp);
                    const float den = wl + ws * E;
                    res = (wl * ol + ws * A) / den;
                    lse = Rp + __logf(den);
                }
                const long long orow = static_cast<long long>(b) * s.Hq + g * G + h;
                a.out[orow * kD + (x % kD)] = __float2bfloat16_rn(res);
                if ((x % kD) == 0) a.lse[orow] = lse;
            }
        }
        asm volatile("bar.sync 1, %0;" ::"r"(kConsumerWarps * 32));
        j0 = j1;
        if (dead) break;
    }
}

struct Plan {
    int n_ctas, max_parts, Cpad;
    size_t off_u, off_wgt, off_R, off_E, off_n, off_done, off_part, off_loco, off_loclam, total;
};

int sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            n = 148;
        if (n <= 0) n = 148;
    }
    return n;
}

Plan make_plan(const Shape& s, int n_sm) {
    Plan p;
    const long long pairs = static_cast<long long>(s.B) * s.Hkv;
    const long long N = pairs * (s.K + 1);
    long long ctas = n_sm;
    if ((N + ctas - 1) / ctas + 1 > kMaxItems) ctas = (N + kMaxItems - 2) / (kMaxItems - 1);
    if (ctas > N) ctas = N;
    p.n_ctas = static_cast<int>(ctas);
    const long long per = N / ctas;                               // every CTA gets per or per+1 items
    p.max_parts = static_cast<int>((s.K + 1 + per - 1) / per) + 1;
    if (p.max_parts > s.K + 1) p.max_parts = s.K + 1;
    p.Cpad = (s.C + 63) / 64 * 64;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = (off + bytes + 255) / 256 * 256; return o; };
    p.off_u = take(sizeof(float) * pairs * p.Cpad);
    p.off_wgt = take(sizeof(float) * pairs * s.G * s.K);
    p.off_R = take(sizeof(float) * pairs * s.G);
    p.off_E = take(sizeof(float) * pairs * s.G);
    p.off_n = take(sizeof(int) * pairs);
    p.off_done = take(sizeof(int) * pairs);
    p.off_part = take(sizeof(float) * pairs * p.max_parts * s.G * kD);
    p.off_loco = take(sizeof(float) * pairs * s.G * kD);
    p.off_loclam = take(sizeof(float) * pairs * s.G);
    p.total = off;
    return p;
}

}  // namespace

bool decode_fast_supports(const Shape& s, int dtype) {
    return dtype == HILS_BF16 && s.is_decode && s.d == kD && s.S == kS && s.W == 1 && s.Hl == s.Hkv && s.G <= 8 &&
           s.K >= 1 && s.K <= 128 && static_cast<long long>(s.B) * s.Hkv * s.T < (1ll << 31) &&
           static_cast<long long>(s.B) * s.Hkv <= 65535;
}

size_t decode_fast_scratch_bytes(const Shape& s) {
    // sized for the largest CTA count the launcher may use, independent of the device queried at run time
    return make_plan(s, 148).total > make_plan(s, 1).total ? make_plan(s, 148).total : make_plan(s, 1).total;
}

int launch_decode_fast(const Shape& s, const Tensors& t, cudaStream_t stream) {
    const Plan p = make_plan(s, 148);
    if (t.scratch_bytes < p.total) return HILS_ERR_WORKSPACE;
    const int pairs = s.B * s.Hkv;
    char* sc = static_cast<char*>(t.scratch);
    DArgs a;
    a.s = s;
    a.q = static_cast<const __nv_bfloat16*>(t.q);
    a.lm = static_cast<const __nv_bfloat16*>(t.landmarks);
    a.bias = t.bias;
    a.seq_lens = t.seq_lens;
    a.out = static_cast<__nv_bfloat16*>(t.out);
    a.lse = t.lse;
    a.sel = t.sel_idx;
    a.status = t.status;
    a.u = reinterpret_cast<float*>(sc + p.off_u);
    a.Cpad = p.Cpad;
    a.wgt = reinterpret_cast<float*>(sc + p.off_wgt);
    a.Rh = reinterpret_cast<float*>(sc + p.off_R);
    a.Eh = reinterpret_cast<float*>(sc + p.off_E);
    a.pair_n = reinterpret_cast<int*>(sc + p.off_n);
    a.done = reinterpret_cast<int*>(sc + p.off_done);
    a.part = reinterpret_cast<float*>(sc + p.off_part);
    a.loc_o = reinterpret_cast<float*>(sc + p.off_loco);
    a.loc_lam = reinterpret_cast<float*>(sc + p.off_loclam);
    a.max_parts = p.max_parts;
    a.n_ctas = p.n_ctas;

    CUtensorMap map_k, map_v;
    const uint64_t rows = static_cast<uint64_t>(pairs) * s.T;
    if (!make_bf16_2d_map(&map_k, t.k, rows, kD, 64, kS) || !make_bf16_2d_map(&map_v, t.v, rows, kD, 64, kS))
        return HILS_ERR_CUDA;

    const size_t attend_smem = kStages * kStageBytes + sizeof(AttendSmem) + 1024;
    static bool attr_done = false;
    if (!attr_done) {
        if (cudaFuncSetAttribute(decode_attend_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(attend_smem)) != cudaSuccess)
            return HILS_ERR_CUDA;
        attr_done = true;
    }

    const int nseg = (s.C + kScoreChunksPerCta - 1) / kScoreChunksPerCta;
    decode_score_kernel<<<dim3(nseg > 0 ? nseg : 1, pairs), kScoreThreads, 0, stream>>>(a);
    if (cudaGetLastError() != cudaSuccess) return HILS_ERR_CUDA;
    trace_mark("decode_score", stream);

    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cfg.gridDim = dim3(pairs);
    cfg.blockDim = dim3(kSelThreads);
    cfg.dynamicSmemBytes = 0;
    if (cudaLaunchKernelEx(&cfg, decode_select_kernel, a) != cudaSuccess) return HILS_ERR_CUDA;
    trace_mark("decode_select", stream);

    cfg.gridDim = dim3(p.n_ctas);
    cfg.blockDim = dim3(kAttendThreads);
    cfg.dynamicSmemBytes = attend_smem;
    if (cudaLaunchKernelEx(&cfg, decode_attend_kernel, map_k, map_v, a) != cudaSuccess) return HILS_ERR_CUDA;
    trace_mark("decode_attend", stream);
    return 3;
}

// ------------------------------------------------------------------------- allocation-free variant
// Scratch for callers that cannot obtain device memory themselves.  The array belongs to the loaded
// library image: every GPU that loads libhils.so carries these 8 MiB until the process exits.
constexpr size_t kNoAllocBytes = 8u << 20;
constexpr int kMaxDevices = 64;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

size_t decode_noalloc_capacity() { return kNoAllocBytes; }

int launch_decode_noalloc(const Shape& s, const Tensors& t_in, int32_t* device_status, cudaStream_t stream) {
    const size_t need = kStatusBytes + decode_fast_scratch_bytes(s);
    if (need > kNoAllocBytes) return HILS_ERR_WORKSPACE;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return HILS_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return HILS_ERR_UNSUPPORTED;
    // In host code `g_noalloc_scratch` is only a handle for the symbol, not an address a kernel can
    // use: the device address is looked up once per device, with that device current.
    static void* dev_ptr[kMaxDevices] = {};
    if (!dev_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return HILS_ERR_CUDA;
        dev_ptr[dev] = p;
    }
    unsigned char* base = static_cast<unsigned char*>(dev_ptr[dev]);
    // The array keeps whatever the previous call left: the status word has to start at zero
    // (the per-pair completion counters are re-zeroed by decode_select on every call).
    if (cudaMemsetAsync(base, 0, kStatusBytes, stream) != cudaSuccess) return HILS_ERR_CUDA;
    Tensors t = t_in;
    t.status = reinterpret_cast<int*>(base);
    t.scratch = base + kStatusBytes;
    t.scratch_bytes = kNoAllocBytes - kStatusBytes;
    const int n = launch_decode_fast(s, t, stream);
    if (n < 0) return n;
    if (device_status &&
        cudaMemcpyAsync(device_status, base, sizeof(int32_t), cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
        return HILS_ERR_CUDA;
    return n;
}

}  // namespace hils
