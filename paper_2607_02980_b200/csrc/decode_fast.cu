// Bandwidth-tuned decode kernels: bf16, d = 128, S = 64, G <= 8, one landmark per KV head, any local window of
// up to 16 chunks (W <= 897).
//
//   decode_score   streams the landmarks of every (sequence, KV head) once with 128-bit loads and
//                  scores them against the G query heads with warp MMA (landmark rows are the A
//                  operand straight from global memory); writes the group score u_c = max_h s^h_c.
//   decode_select  one CTA per (sequence, KV head): exact top-K of u (ties to the lower chunk id) by radix
//                  selection on the ordered score keys (8 bits per pass over keys cached in shared memory),
//                  ascending ids, then the per-head surrogate scores of the selected chunks and the
//                  fusion weights exp(s^h_c - max_c s^h_c).
//   decode_attend  persistent CTAs over a flat list of (pair, slot) items; K/V chunks arrive through
//                  a TMA + mbarrier ring (128B-swizzled tiles), each consumer warp runs one chunk at
//                  a time: QK^T, the chunk's own softmax, PV (Eq. HiLS weights); the CTA that
//                  finishes a pair last mixes the partial sums with the local branch (App. C).
#include "internal.h"
#include "tma.cuh"
// Timeline instrumentation, compiled only with -DX_STAMP (never in the library that is shipped): the kernels record
// globaltimer stamps of their phases (even slots: earliest, odd slots: latest over the CTAs), hils_debug_stamps reads
// them back.  The timelines quoted in the kernels' comments come from such builds.
#ifdef X_STAMP
namespace hils { __device__ unsigned long long g_dbg[16]; }
__device__ __forceinline__ unsigned long long gtime() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#define STAMP_MIN(i) if (threadIdx.x == 0) atomicMin(&hils::g_dbg[i], gtime())
#define STAMP_MAX(i) if (threadIdx.x == 0) atomicMax(&hils::g_dbg[i], gtime())
extern "C" void hils_debug_stamps(unsigned long long* out, int reset) {
    unsigned long long h[16];
    cudaMemcpyFromSymbol(h, hils::g_dbg, sizeof(h));
    for (int i = 0; i < 16; ++i) out[i] = h[i];
    if (reset) { for (int i = 0; i < 16; ++i) h[i] = (i & 1) ? 0ull : ~0ull; cudaMemcpyToSymbol(hils::g_dbg, h, sizeof(h)); }
}
#else
#define STAMP_MIN(i)
#define STAMP_MAX(i)
#endif

namespace hils {
namespace {

constexpr int kD = 128;
constexpr int kS = 64;
constexpr int kScoreThreads = 256;
constexpr int kScoreChunksPerCta = 256;      // 8 warps x 2 iterations x 16 chunks
constexpr int kStages = 6;
constexpr int kStageBytes = 2 * kS * kD * 2; // K tile + V tile
constexpr int kMaxItems = 1024;
constexpr int kConsumerWarps = 6;       // == kStages: a stage is always consumed by the same warp, so no
                                        // waiter can ever be more than one mbarrier phase away from its stage
static_assert(kStages % kConsumerWarps == 0, "stage ownership must be fixed per consumer warp");
constexpr int kAttendThreads = (kConsumerWarps + 1) * 32;
constexpr float kLog2e = 1.4426950408889634f;

struct DArgs {
    Shape s;
    const __nv_bfloat16* q;
    const __nv_bfloat16* q_route;  // routing query for the surrogate scores (= q unless a separate one was given)
    const __nv_bfloat16* lm;
    const float* bias;
    const int32_t* seq_lens;
    __nv_bfloat16* out;
    float* lse;
    int32_t* sel;
    int* status;
    // scratch
    float* u;          // [pairs, Cpad] group scores
    float* uh;         // [pairs, G, Cpad] per-head scores (written by the streaming scoring kernel), or NULL
    int Cpad;
    float* wgt;        // [pairs, G, K] exp(s^h_c - R_h) of the selected chunks
    float* Rh;         // [pairs, G]    max_c s^h_c over the selected chunks
    float* Eh;         // [pairs, G]    sum of wgt
    int* pair_n;       // [pairs]       number of selected chunks, -1 = invalid sequence length
    int* done;         // [pairs]       slots finished (zeroed by the selection)
    float* part;       // [pairs, max_parts, G, 128] weighted partial sums
    float* loc_o;      // [pairs, NL, G, 128] outputs of the chunks of the local window (NL = max_local_slots(W))
    float* loc_lam;    // [pairs, NL, G]      their log masses (together: log Z_swa)
    int max_parts;
    int n_ctas;
    const int32_t* block_table;   // paged caches: [B, C] page of every logical chunk, or NULL (contiguous caches)
    int num_pages;
};

// The local window [l(i), i] of the query at i = seq_len - 1 (Sec. 2.1) is whole chunks plus the causal part of the
// query's own chunk: chunks lc .. ci, at most max_local_slots(W) of them.  Each is attended like a selected chunk,
// with its own softmax; its mass is the exact log-sum-exp of its scores, so mixing by the masses reproduces the
// single softmax over the window (Eq. chunk mass).  Candidates for selection are the chunks 0 .. lc - 1.
__host__ __device__ inline int max_local_slots(int W) { return (W - 1 + kS - 1) / kS + 1; }
// Multi-token decode: query b of the call sees the cache of sequence b / qps up to and including its own token.
__device__ __forceinline__ int query_seq_len(const DArgs& a, int b) {
    const int q = a.s.qps;
    return q == 1 ? a.seq_lens[b] : a.seq_lens[b / q] - (q - 1) + b % q;
}
__device__ __forceinline__ int first_local_chunk(int seq, int W) { return local_lo(seq - 1, W, kS) / kS; }

// ------------------------------------------------------------------------------------------ select
// Exact top-K by radix selection on the ordered score keys, one CTA per (sequence, KV head) pair.  The K-th best key T
// is found digit by digit (four passes of 8 bits, most significant first): every pass histograms the digit of the
// candidates that still match the prefix found so far (one private histogram per warp: equal digits are the rule in
// the leading, exponent, byte), sums the histograms and walks the 256 bins from the top until K candidates are
// covered.  Chunks with a key above T are selected; of those equal to T as many as are still missing, lowest chunk ids
// first -- if there are more than that, a second selection of the same kind runs on their ids.  The keys are cached
// in shared memory after the first pass (they come from L2) when they fit.  Integer arithmetic throughout: exact and
// independent of the thread count.
//
// A pass over the list costs its instructions, not its bytes (one SM works on a pair's whole list), so lists of up to
// 16 candidates per thread take a shorter way first (select_in_registers): every thread keeps its scores in
// registers; the span between the smallest and the largest score is cut into 2048 equal bins (equal in value: the
// bins of a radix digit are equal in the exponent, and most scores of a list share two or three exponents, which
// serialises their counter updates), one histogram pass and one scan find the bin the K-th best score falls into,
// everything above it is selected and the bin's members are ranked against each other directly by (key, then lower
// chunk id).  A bin with more than kSelTieCap members (massive ties) falls back to the passes described above.
constexpr int kSelMaxK = 128;
constexpr int kSelMaxWarps = 32;
constexpr int kSelKeyCap = 40960;            // keys cached in shared memory (160 KB); longer lists re-read the scores
constexpr int kSelTieCap = 512;              // candidates of the boundary bin that are ranked directly
constexpr int kSelRegKeys = 16;              // keys a thread holds in registers on the short way
constexpr int kSelBins = 2048;               // counters of the short way's histogram (at most: about half a bin per candidate)

struct SelState {
    int hist[256];                           // summed histogram of the current pass
    unsigned prefix, mask;                   // digits fixed so far
    int remaining;                           // how many candidates matching the prefix are still wanted from the top
    int equal;                               // candidates whose key equals the finished prefix
    int nout;                                // selected so far
    int ntie, bstar, above;                  // short way: the bin of the K-th best score
    unsigned kmin, kmax;                     // short way: span of the scores (ordered keys)
    int wsum[kSelMaxWarps];
};

// One selection: the `want`-th largest value of val(i) over the candidates i in [0, n) for which live(i) holds
// (bits [top_bit, 0] are examined, 8 at a time).  Returns the value; `equal` = how many live candidates hold exactly
// that value, `remaining` = how many of those are wanted.  Called by every thread of the CTA.
template <typename Val, typename Live>
__device__ unsigned radix_kth(SelState& st, int (*whist)[256], int n, int want, int top_shift, Val val, Live live,
                          bool first_hist_ready = false) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, NT = blockDim.x, nw = NT >> 5;
    if (tid == 0) { st.prefix = 0u; st.mask = 0u; st.remaining = want; }
    if (!first_hist_ready)
        for (int x = lane; x < 256; x += 32) whist[warp][x] = 0;
    __syncthreads();
    for (int shift = top_shift; shift >= 0; shift -= 8) {
        const unsigned prefix = st.prefix, mask = st.mask;
        if (!(first_hist_ready && shift == top_shift)) {
            for (int i = tid; i < n; i += NT) {
                if (!live(i)) continue;
                const unsigned v = val(i);
                if ((v & mask) == prefix) atomicAdd(&whist[warp][(v >> shift) & 255u], 1);
            }
        }
        __syncthreads();
        // sum of the warps' histograms (left zeroed for the next pass)
        for (int x = tid; x < 256; x += NT) {
            int sum = 0;
#pragma unroll 8
            for (int w = 0; w < nw; ++w) { sum += whist[w][x]; whist[w][x] = 0; }
            st.hist[x] = sum;
        }
        __syncthreads();
        if (warp == 0) {
            // lane l owns bins 255 - 8 l .. 248 - 8 l; the digit is the highest bin d with count(bins >= d) >= remaining
            const int rem = st.remaining;
            int h8[8];
            int tsum = 0;
#pragma unroll
            for (int x = 0; x < 8; ++x) { h8[x] = st.hist[255 - 8 * lane - x]; tsum += h8[x]; }
            int inc = tsum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int nn = __shfl_up_sync(kFullMask, inc, o);
                if (lane >= o) inc += nn;
            }
            int cum = inc - tsum;
            if (cum < rem && inc >= rem) {          // exactly one lane
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    if (cum < rem && cum + h8[x] >= rem) {
                        st.prefix = prefix | (static_cast<unsigned>(255 - 8 * lane - x) << shift);
                        st.mask = mask | (255u << shift);
                        st.remaining = rem - cum;
                        st.equal = h8[x];
                    }
                    cum += h8[x];
                }
            }
        }
        __syncthreads();
    }
    return st.prefix;
}

struct SelShared {
    int sel_s[kSelMaxK];
    int raw_s[kSelMaxK];                     // selected ids in arrival order
    float lam_s[8][kSelMaxK];
    alignas(16) __nv_bfloat16 q_s[8][kD + 8];
    SelState st;
};
constexpr size_t kSelLmBytes = 64 * (kD + 8) * 2;          // staged landmark rows alias the selection buffers
// dynamic shared memory of the selection: per-warp histograms, then the cached keys
// dynamic shared memory of the selection: histograms (nw of 256 counters, or the short way's 2048), then the cached
// keys or the short way's boundary-bin members
__host__ __device__ inline size_t sel_hist_ints(int nw) { return nw * 256 > kSelBins ? nw * 256 : kSelBins; }
__host__ __device__ inline size_t sel_dyn_bytes(int nw, int ncached) {
    const size_t keys = static_cast<size_t>(ncached) * sizeof(unsigned), ties = static_cast<size_t>(kSelTieCap) * 2 * sizeof(unsigned);
    const size_t need = sel_hist_ints(nw) * sizeof(int) + (keys > ties ? keys : ties);
    return need > kSelLmBytes ? need : kSelLmBytes;
}

// Walks the `nbins` counters of hist from the top bin down and finds the bin in which the running count reaches
// `need`: st.bstar = that bin, st.above = candidates in the bins above it, st.equal = candidates in it.  Called by
// every thread; ends with a barrier.
__device__ void scan_from_top(SelState& st, const int* hist, int nbins, int need) {
    // (a step of a few instructions: with every warp of a large CTA taking part it would cost their issue slots, so
    //  at most 256 threads walk the bins)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, NT = blockDim.x < 256 ? blockDim.x : 256, nw = NT >> 5;
    if (tid >= NT) { __syncthreads(); __syncthreads(); __syncthreads(); return; }
    const int per = nbins > NT ? nbins / NT : 1;          // nbins and NT are powers of two
    int mine = 0;
    for (int x = 0; x < per; ++x) {
        const int bk = nbins - 1 - (tid * per + x);
        if (bk >= 0) mine += hist[bk];
    }
    int inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int nn = __shfl_up_sync(kFullMask, inc, o);
        if (lane >= o) inc += nn;
    }
    if (lane == 31) st.wsum[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const int tot = lane < nw ? st.wsum[lane] : 0;
        int acc = tot;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int nn = __shfl_up_sync(kFullMask, acc, o);
            if (lane >= o) acc += nn;
        }
        if (lane < nw) st.wsum[lane] = acc - tot;          // candidates in the bins of the warps before this one
    }
    __syncthreads();
    int cum = st.wsum[warp] + inc - mine;                  // candidates in the bins above this thread's
    if (cum < need && cum + mine >= need) {                // exactly one thread
        for (int x = 0; x < per; ++x) {
            const int bk = nbins - 1 - (tid * per + x);
            const int h = bk >= 0 ? hist[bk] : 0;
            if (cum < need && cum + h >= need) { st.bstar = bk; st.above = cum; st.equal = h; }
            cum += h;
        }
    }
    __syncthreads();
}

// Exact top-`want` of the n <= kSelRegKeys * blockDim.x scores u[0 .. n) (see above).  hist: kSelBins counters;
// tie_k / tie_i: kSelTieCap entries each.  Returns true with the selected candidate ids in raw_s[0 .. want) (any
// order); false, with nothing written that matters, when the bin of the K-th best score holds more than kSelTieCap
// candidates (or the scores have no span).  Called by every thread.
__device__ bool select_in_registers(SelState& st, int* hist, const float* u, int n, int want, int* raw_s,
                                    unsigned* tie_k, int* tie_i) {
    const int tid = threadIdx.x, lane = tid & 31, NT = blockDim.x;
    float v[kSelRegKeys];
#pragma unroll
    for (int x = 0; x < kSelRegKeys; ++x) {
        const int i = x * NT + tid;
        v[x] = i < n ? __ldcg(u + i) : 0.f;
    }
    // about two candidates per bin: the bin of the K-th best score then holds a handful, and short lists do not pay
    // for zeroing and walking counters they cannot fill
    int nbins = 256;
    while (nbins < kSelBins && 2 * nbins < n) nbins <<= 1;
    for (int x = tid; x < nbins; x += NT) hist[x] = 0;
    if (tid == 0) { st.nout = 0; st.ntie = 0; st.kmin = 0xffffffffu; st.kmax = 0u; }
    __syncthreads();
    // span of the scores
    unsigned kmin = 0xffffffffu, kmax = 0u;
#pragma unroll
    for (int x = 0; x < kSelRegKeys; ++x) {
        if (x * NT + tid < n) {
            const unsigned k = ordered_key(v[x]);
            kmin = min(kmin, k);
            kmax = max(kmax, k);
        }
    }
    kmin = __reduce_min_sync(kFullMask, kmin);
    kmax = __reduce_max_sync(kFullMask, kmax);
    if (lane == 0) { atomicMin(&st.kmin, kmin); atomicMax(&st.kmax, kmax); }
    __syncthreads();
    const float lo = key_to_float(st.kmin), hi = key_to_float(st.kmax);
    const float inv = static_cast<float>(nbins) / (hi - lo);
    // (no span, or a span that is not a number: every candidate would land in one bin)
    if (!(hi > lo) || !(inv > 0.f) || !(inv < INFINITY)) return false;
    // bin of a score: the same expression wherever it is needed, non-decreasing in the score
    auto bin_of = [&](float x) { return min(nbins - 1, max(0, static_cast<int>((x - lo) * inv))); };
#pragma unroll
    for (int x = 0; x < kSelRegKeys; ++x)
        if (x * NT + tid < n) atomicAdd(&hist[bin_of(v[x])], 1);
    __syncthreads();
    scan_from_top(st, hist, nbins, want);
    const int bstar = st.bstar, above = st.above, m = st.equal;
    if (m > kSelTieCap) return false;
#pragma unroll
    for (int x = 0; x < kSelRegKeys; ++x) {
        const int i = x * NT + tid;
        if (i < n) {
            const int bk = bin_of(v[x]);
            if (bk > bstar) {
                raw_s[atomicAdd(&st.nout, 1)] = i;
            } else if (bk == bstar) {
                const int pos = atomicAdd(&st.ntie, 1);
                tie_k[pos] = ordered_key(v[x]);
                tie_i[pos] = i;
            }
        }
    }
    __syncthreads();
    // the `need` best of the bin's m members: rank = members ahead of mine (higher key, or the same key and a lower
    // chunk id); eight lanes share a member
    const int need = want - above;
    for (int e0 = 0; e0 < m; e0 += NT / 8) {
        const int e = e0 + (tid >> 3), part = tid & 7;
        if (e0 + ((tid >> 5) << 2) >= m) continue;          // none of this warp's four members exists (warp-uniform)
        const unsigned ke = e < m ? tie_k[e] : 0u;
        const int ie = e < m ? tie_i[e] : 0;
        int rank = 0;
        for (int f = part; f < m; f += 8) {
            const unsigned kf = tie_k[f];
            rank += (kf > ke || (kf == ke && tie_i[f] < ie)) ? 1 : 0;
        }
        rank += __shfl_xor_sync(kFullMask, rank, 1);
        rank += __shfl_xor_sync(kFullMask, rank, 2);
        rank += __shfl_xor_sync(kFullMask, rank, 4);
        if (e < m && part == 0 && rank < need) raw_s[above + rank] = ie;
    }
    __syncthreads();
    return true;
}

// Ascending chunk ids: position = number of selected ids below mine (eight lanes share an element).  Called by every
// thread; ends with a barrier.
__device__ void sort_ids_ascending(const int* raw_s, int* sel_s, int n) {
    const int tid = threadIdx.x, NT = blockDim.x;
    for (int t0 = 0; t0 < n; t0 += NT / 8) {
        const int t = t0 + (tid >> 3), part = tid & 7;
        if (t0 + ((tid >> 5) << 2) >= n) continue;           // none of this warp's four elements exists (warp-uniform)
        const int idt = t < n ? raw_s[t] : 0;
        int pos = 0;
        for (int j = part; j < n; j += 8) pos += raw_s[j] < idt ? 1 : 0;
        pos += __shfl_xor_sync(kFullMask, pos, 1);
        pos += __shfl_xor_sync(kFullMask, pos, 2);
        pos += __shfl_xor_sync(kFullMask, pos, 4);
        if (t < n && part == 0) sel_s[pos] = idt;
    }
    __syncthreads();
}

// Exact top-K of the group scores of one (sequence, KV head) pair (ties: lower chunk id), ascending ids,
// then the per-head surrogate scores of the selected chunks and the fusion weights.  Called by every
// thread of the pair's CTA (nw warps); dyn: nw histograms of 256 counters, then room for the cached keys.
__device__ void select_pair(const DArgs& a, int pair, int ncand, SelShared& sh, uint8_t* dyn, int nw) {
    const Shape& s = a.s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int NT = nw * 32;
    const int b = pair / s.Hkv, g = pair % s.Hkv;
    const int K = s.K, G = s.G;
    int32_t* sel = a.sel + static_cast<long long>(pair) * K;
    const int n = min(K, ncand);
    const float* u = a.u + static_cast<long long>(pair) * a.Cpad;
    int* sel_s = sh.sel_s;
    int (*whist)[256] = reinterpret_cast<int (*)[256]>(dyn);
    unsigned* keys = reinterpret_cast<unsigned*>(dyn + sel_hist_ints(nw) * sizeof(int));
    // room for the keys was requested at launch only if the longest possible list fits (see launch_decode_fast)
    const bool cached = (s.T - 1) / kS < kSelKeyCap;

    if (ncand <= K) {
        for (int t = tid; t < K; t += NT) sel_s[t] = t < ncand ? t : -1;
        __syncthreads();
    } else if (ncand <= kSelRegKeys * NT &&
               select_in_registers(sh.st, reinterpret_cast<int*>(dyn), u, ncand, K, sh.raw_s, keys,
                                   reinterpret_cast<int*>(keys + kSelTieCap))) {
        sort_ids_ascending(sh.raw_s, sel_s, n);
    } else {
        if (cached) {
            // the scores come from L2: sixteen loads in flight per thread; the histogram of the keys' leading byte
            // (the first selection pass) is taken on the way
            for (int x = tid & 31; x < 256; x += 32) whist[tid >> 5][x] = 0;
            __syncwarp();
            for (int i0 = 0; i0 < ncand; i0 += 16 * NT) {
                float v[16];
#pragma unroll
                for (int x = 0; x < 16; ++x) {
                    const int i = i0 + x * NT + tid;
                    v[x] = i < ncand ? __ldcg(u + i) : 0.f;
                }
#pragma unroll
                for (int x = 0; x < 16; ++x) {
                    const int i = i0 + x * NT + tid;
                    if (i < ncand) {
                        const unsigned k = ordered_key(v[x]);
                        keys[i] = k;
                        atomicAdd(&whist[tid >> 5][k >> 24], 1);
                    }
                }
            }
            __syncthreads();
        }
        auto key_of = [&](int i) { return cached ? keys[i] : ordered_key(__ldcg(u + i)); };
        // T = the K-th best score key; `quota` of the chunks that hold exactly T are still wanted
        const unsigned T = radix_kth(sh.st, whist, ncand, K, 24, key_of, [](int) { return true; }, cached);
        const int quota = sh.st.remaining, equal = sh.st.equal;
        __syncthreads();
        // more ties than places: the `quota` lowest chunk ids among them, i.e. the quota-th largest of ~id
        unsigned idcut = 0u;                      // chunks with key == T and ~id >= idcut are taken
        if (equal > quota) {
            idcut = radix_kth(sh.st, whist, ncand, quota, 16, [](int i) { return 0x00ffffffu - static_cast<unsigned>(i); },
                              [&](int i) { return key_of(i) == T; });
            __syncthreads();
        }
        if (tid == 0) sh.st.nout = 0;
        __syncthreads();
        for (int i = tid; i < ncand; i += NT) {
            const unsigned k = key_of(i);
            if (k > T || (k == T && 0x00ffffffu - static_cast<unsigned>(i) >= idcut)) {
                const int pos = atomicAdd(&sh.st.nout, 1);
                if (pos < kSelMaxK) sh.raw_s[pos] = i;
            }
        }
        __syncthreads();
        sort_ids_ascending(sh.raw_s, sel_s, n);
    }
    for (int t = tid; t < K; t += NT) sel[t] = t < n ? sel_s[t] : -1;
    // --- per-head surrogate scores of the selected chunks and the fusion weights: the selected
    //     landmark rows and the G queries are staged in shared memory with one round of 16-byte
    //     loads, then every thread computes (chunk, head) dot products
    if (a.uh) {
        // the scoring kernel left every head's scores behind: pick the selected chunks' out of that table
        for (int x = tid; x < n * G; x += NT) {
            const int t = x / G, h = x % G;
            sh.lam_s[h][t] = __ldcg(a.uh + (static_cast<long long>(pair) * G + h) * a.Cpad + sel_s[t]);
        }
    } else {
    __nv_bfloat16 (*lm_s)[kD + 8] = reinterpret_cast<__nv_bfloat16 (*)[kD + 8]>(dyn);
    const int per = s.Hl / s.Hkv;                        // landmark rows per chunk: 1, or one per query head (G)
    const long long lrow0 = (static_cast<long long>(b / s.qps) * s.Hl + g * per) * s.C;      // landmark head 0 of this KV head
    const __nv_bfloat16* qg = a.q_route + (static_cast<long long>(b) * s.Hq + g * G) * kD;     // fusion scores: q-hat
    for (int x = tid; x < G * 16; x += NT)
        *reinterpret_cast<uint4*>(&sh.q_s[x >> 4][(x & 15) * 8]) = *reinterpret_cast<const uint4*>(qg + (x >> 4) * kD + (x & 15) * 8);
    const int tstep = 64 / per;                          // selected chunks staged per round (64 landmark rows)
    for (int t0 = 0; t0 < n; t0 += tstep) {
        const int nt = min(tstep, n - t0);
        __syncthreads();
        // staged row (t * per + hh): landmark head hh of selected chunk t0 + t
        for (int x0 = 0; x0 < nt * per * 16; x0 += 4 * NT) {       // four 16-byte loads in flight per thread
            uint4 v[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int x = x0 + r * NT + tid;
                if (x < nt * per * 16) {
                    const int row = x >> 4, tt = row / per, hh = row % per;
                    v[r] = *reinterpret_cast<const uint4*>(a.lm + (lrow0 + static_cast<long long>(hh) * s.C + sel_s[t0 + tt]) * kD + (x & 15) * 8);
                }
            }
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int x = x0 + r * NT + tid;
                if (x < nt * per * 16) *reinterpret_cast<uint4*>(&lm_s[x >> 4][(x & 15) * 8]) = v[r];
            }
        }
        __syncthreads();
        for (int x = tid; x < nt * G; x += NT) {
            const int t = x / G, h = x % G;
            const int hh = per == 1 ? 0 : h;             // the landmark head this query head scores against
            const __nv_bfloat16* lr = lm_s[t * per + hh];
            const __nv_bfloat16* qr = sh.q_s[h];
            float acc = 0.f;
#pragma unroll 8
            for (int e = 0; e < kD; e += 2) {
                const float2 lv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(lr + e));
                const float2 qv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(qr + e));
                acc = fmaf(lv.x, qv.x, acc);
                acc = fmaf(lv.y, qv.y, acc);
            }
            const float bb = a.bias ? a.bias[lrow0 + static_cast<long long>(hh) * s.C + sel_s[t0 + t]] : 0.f;
            sh.lam_s[h][t0 + t] = acc * s.scale + bb;
        }
    }
    }
    __syncthreads();
    for (int h = warp; h < G; h += nw) {
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
    const int seq = query_seq_len(a, b);
    STAMP_MIN(0);
    if (seq < 1 || seq > s.T) return;
    const int ncand = first_local_chunk(seq, s.W);
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
        const __nv_bfloat16* qrow = a.q_route + (static_cast<long long>(b) * s.Hq + g * s.G + gq) * kD;
#pragma unroll
        for (int kb = 0; kb < 4; ++kb) qf[kb] = *reinterpret_cast<const uint4*>(qrow + kb * 32 + t * 8);
    }
    // One landmark per KV head (per = 1: all heads score the same row), or one per query head (per = G, App. C:
    // k'_c in R^{G x d}): then head hh scores only its own landmark row and only column hh of the MMA is kept.
    const int per = s.Hl / s.Hkv;
    float* u = a.u + static_cast<long long>(pair) * a.Cpad;
    int c0[2];
    float best[2][2];
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        c0[it] = c_begin + (warp * 2 + it) * 16;
        best[it][0] = best[it][1] = -INFINITY;
    }
    for (int hh = 0; hh < per; ++hh) {
        const long long lrow = (static_cast<long long>(b / s.qps) * s.Hl + g * per + hh) * s.C;
        const __nv_bfloat16* lm = a.lm + lrow * kD;
        const float* bias = a.bias ? a.bias + lrow : nullptr;
        uint4 x[2][2][4];
#pragma unroll
        for (int it = 0; it < 2; ++it) {
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
            const bool h0 = per == 1 ? 2 * t < s.G : 2 * t == hh, h1 = per == 1 ? 2 * t + 1 < s.G : 2 * t + 1 == hh;
            float m0 = fmaxf(h0 ? acc[0] : -INFINITY, h1 ? acc[1] : -INFINITY);
            float m1 = fmaxf(h0 ? acc[2] : -INFINITY, h1 ? acc[3] : -INFINITY);
            m0 = fmaxf(m0, __shfl_xor_sync(kFullMask, m0, 1));
            m1 = fmaxf(m1, __shfl_xor_sync(kFullMask, m1, 1));
            m0 = fmaxf(m0, __shfl_xor_sync(kFullMask, m0, 2));
            m1 = fmaxf(m1, __shfl_xor_sync(kFullMask, m1, 2));
            const int ca = c0[it] + gq, cb = ca + 8;
            best[it][0] = fmaxf(best[it][0], m0 * s.scale + ((bias && ca < ncand) ? bias[ca] : 0.f));
            best[it][1] = fmaxf(best[it][1], m1 * s.scale + ((bias && cb < ncand) ? bias[cb] : 0.f));
        }
    }
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        const int ca = c0[it] + gq, cb = ca + 8;
        if (t == 0 && ca < ncand) u[ca] = best[it][0];
        if (t == 1 && cb < ncand) u[cb] = best[it][1];
    }
    STAMP_MAX(1);
    pdl_launch_dependents();
}

// The same scores from a persistent kernel that streams the landmark rows through a TMA ring (one landmark row per KV
// head: Hl = Hkv).  decode_score_kernel above runs 2048 short CTAs that each request their 64 KB, wait, compute and
// leave: the bytes in flight drop to zero between a CTA's loads and its successor's.  Here one CTA per SM keeps
// kScStages tiles of 64 landmark rows (16 KB each) requested at all times; the valid tiles of all (sequence, KV head)
// pairs form one list that is cut into equal contiguous ranges, a tile is scored by the warp that owns its stage
// (landmark rows as the B operand of the warp-level MMA, the G query heads in the A rows), the maximum over the heads
// is taken with shuffles and the 64 group scores are written.
constexpr int kScStages = 12;
constexpr int kScStageBytes = kS * kD * 2;
constexpr int kScWarps = 6;                // consumer warps: a stage is always consumed by the same warp
constexpr int kScThreads = (kScWarps + 1) * 32;
constexpr int kScMaxPairs = 4096;            // prefix of the pairs' tile counts in shared memory
static_assert(kScStages % kScWarps == 0, "stage ownership must be fixed per consumer warp");

struct ScoreSmem {
    uint64_t full[kScStages];
    uint64_t empty[kScStages];
    int pref[kScMaxPairs + 1];               // tiles of the pairs before pair p
    int wsum[kScThreads / 32];
    int dead;
};

__global__ void __launch_bounds__(kScThreads, 1)
decode_score_stream_kernel(const __grid_constant__ CUtensorMap map_lm, const DArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    ScoreSmem& sm = *reinterpret_cast<ScoreSmem*>(ring + kScStages * kScStageBytes);
    const Shape& s = a.s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int pairs = s.B * s.Hkv;
    STAMP_MIN(0);
    if (tid == 0) {
        for (int i = 0; i < kScStages; ++i) { mbar_init(&sm.full[i], 1); mbar_init(&sm.empty[i], 1); }
        mbar_fence_init();
        sm.dead = 0;
        sm.pref[0] = 0;
        tma_prefetch_desc(&map_lm);
    }
    __syncthreads();
    // tiles of 64 candidates per pair (0 for an invalid length), inclusive scan over the pairs
    auto pair_ncand = [&](int pr) {
        const int seq = query_seq_len(a, pr / s.Hkv);
        return (seq < 1 || seq > s.T) ? 0 : first_local_chunk(seq, s.W);
    };
    // (thread t sums the tile counts of its pairs [t ppt, (t + 1) ppt), one scan over the threads, then each thread
    //  writes its pairs' entries: two barriers whatever the number of pairs)
    {
        const int ppt = (pairs + kScThreads - 1) / kScThreads;
        const int p_begin = min(pairs, tid * ppt), p_end = min(pairs, p_begin + ppt);
        int mine = 0;
        for (int pr = p_begin; pr < p_end; ++pr) mine += (pair_ncand(pr) + kS - 1) / kS;
        int inc = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int nn = __shfl_up_sync(kFullMask, inc, o);
            if (lane >= o) inc += nn;
        }
        if (lane == 31) sm.wsum[warp] = inc;
        __syncthreads();
        int run = inc - mine;
        for (int w = 0; w < warp; ++w) run += sm.wsum[w];
        for (int pr = p_begin; pr < p_end; ++pr) {
            run += (pair_ncand(pr) + kS - 1) / kS;
            sm.pref[pr + 1] = run;
        }
        __syncthreads();
    }
    const long long total = sm.pref[pairs];
    const int lo = static_cast<int>(total * blockIdx.x / gridDim.x), hi = static_cast<int>(total * (blockIdx.x + 1) / gridDim.x);
    // pair of the range's first tile: last p with pref[p] <= lo
    int p_lo = 0;
    {
        int l = 0, r = pairs;                     // invariant: pref[l] <= lo < pref[r] (when lo < total)
        while (r - l > 1) {
            const int m = (l + r) >> 1;
            if (sm.pref[m] <= lo) l = m; else r = m;
        }
        p_lo = l;
    }
    if (hi > lo) {
        if (warp == kScWarps) {
            // ------------------------------------------------------------------ producer (one lane)
            if (lane == 0) {
                int pr = p_lo;
                for (int x = lo; x < hi; ++x) {
                    while (sm.pref[pr + 1] <= x) ++pr;
                    const int k = x - lo, st = k % kScStages;
                    if (k >= kScStages && !mbar_wait(&sm.empty[st], ((k / kScStages) - 1) & 1)) {
                        set_status(a.status, kDevTimeout);
                        atomicExch(&sm.dead, 1);
                        break;
                    }
                    const int b = pr / s.Hkv, g = pr % s.Hkv;
                    const int row = ((b / s.qps) * s.Hl + g) * s.C + (x - sm.pref[pr]) * kS;
                    uint8_t* dst = ring + st * kScStageBytes;
                    mbar_expect_tx(&sm.full[st], kScStageBytes);
                    tma_load_2d(dst, &map_lm, &sm.full[st], 0, row);
                    tma_load_2d(dst + 8192, &map_lm, &sm.full[st], 64, row);
                }
            }
        } else {
            // ------------------------------------------------------------------ consumers
            const int gq = lane >> 2, t = lane & 3;
            int pr = p_lo, cur = -1;
            uint32_t aq[8][2];
            for (int x = lo + warp; x < hi; x += kScWarps) {
                while (sm.pref[pr + 1] <= x) ++pr;
                const int b = pr / s.Hkv, g = pr % s.Hkv;
                if (pr != cur) {
                    cur = pr;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) { aq[ks][0] = 0u; aq[ks][1] = 0u; }
                    if (gq < s.G) {
                        const __nv_bfloat16* qrow = a.q_route + (static_cast<long long>(b) * s.Hq + g * s.G + gq) * kD;
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            aq[ks][0] = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 2 * t);
                            aq[ks][1] = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8 + 2 * t);
                        }
                    }
                }
                const int k = x - lo, st = k % kScStages;
                if (!mbar_wait(&sm.full[st], (k / kScStages) & 1)) {
                    if (lane == 0) { set_status(a.status, kDevTimeout); atomicExch(&sm.dead, 1); }
                    break;
                }
                // D[chunk][head] = landmark rows (A, 16 chunks per tile of the MMA, straight from the swizzled stage) x q^T
                // (B: the G heads in the columns): every A row is a chunk, and the maximum over the heads is a maximum
                // over a thread's own two columns and its neighbours'
                const uint32_t lm_addr = smem_u32(ring + st * kScStageBytes);
                float acc[4][4];
#pragma unroll
                for (int mt = 0; mt < 4; ++mt) {
                    acc[mt][0] = acc[mt][1] = acc[mt][2] = acc[mt][3] = 0.f;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const int row = mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                        const int dim = ks * 16 + (lane >> 4) * 8;
                        uint32_t fr[4];
                        ldmatrix_x4(lm_addr + (dim >> 6) * 8192 + swz128(row, (dim & 63) >> 3), fr[0], fr[1], fr[2], fr[3]);
                        mma_bf16_16816(acc[mt], fr, aq[ks][0], aq[ks][1]);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.empty[st]);
                // acc[mt][0..1]: chunk c0 + 16 mt + gq, heads 2 t, 2 t + 1; acc[mt][2..3]: chunk + 8
                const int c0 = (x - sm.pref[pr]) * kS;
                const int ncand = pair_ncand(pr);
                const float* bias = a.bias ? a.bias + (static_cast<long long>(b / s.qps) * s.Hl + g) * s.C : nullptr;
                float* u = a.u + static_cast<long long>(pr) * a.Cpad;
                float* uh0 = a.uh + (static_cast<long long>(pr) * s.G + 2 * t) * a.Cpad;       // head 2 t (2 t + 1: + Cpad)
                const bool h0 = 2 * t < s.G, h1 = 2 * t + 1 < s.G;
#pragma unroll
                for (int mt = 0; mt < 4; ++mt) {
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        const int c = c0 + mt * 16 + half * 8 + gq;
                        const float bb = (bias && c < ncand) ? bias[c] : 0.f;
                        const float s0 = acc[mt][2 * half] * s.scale + bb, s1 = acc[mt][2 * half + 1] * s.scale + bb;
                        // the head's own scores: the mixing logits of whatever chunks get selected (Eq. HiLS weights)
                        if (c < ncand) {
                            if (h0) uh0[c] = s0;
                            if (h1) uh0[a.Cpad + c] = s1;
                        }
                        float m = fmaxf(h0 ? s0 : -INFINITY, h1 ? s1 : -INFINITY);
                        m = fmaxf(m, __shfl_xor_sync(kFullMask, m, 1));
                        m = fmaxf(m, __shfl_xor_sync(kFullMask, m, 2));
                        if (t == 0 && c < ncand) u[c] = m;
                    }
                }
            }
        }
    }
    STAMP_MAX(1);
    pdl_launch_dependents();
}

// One CTA per (sequence, KV head) pair: 4 warps for candidate lists of up to 1024 chunks, 8 up to 4096, else 32.
// Dynamic shared memory: sel_dyn_bytes.
__global__ void __launch_bounds__(kSelMaxWarps * 32) decode_select_kernel(const DArgs a) {
    __shared__ SelShared sh;
    extern __shared__ __align__(16) uint8_t sel_dyn[];
    const Shape& s = a.s;
    const int pair = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
    const int b = pair / s.Hkv, g = pair % s.Hkv;
    const int seq = query_seq_len(a, b);
    STAMP_MIN(2);
    pdl_wait();                                        // the previous kernels' reads and writes of the scratch are over
    STAMP_MIN(4);
    if (seq < 1 || seq > s.T) {
        // invalid length: flag it, emit empty outputs
        if (tid == 0) { set_status(a.status, kDevBadIndex); a.pair_n[pair] = -1; a.done[pair] = 0; }
        for (int t = tid; t < s.K; t += nt) a.sel[static_cast<long long>(pair) * s.K + t] = -1;
        for (int x = tid; x < s.G * kD; x += nt)
            a.out[(static_cast<long long>(b) * s.Hq + g * s.G) * kD + x] = __float2bfloat16_rn(0.f);
        if (tid < s.G) a.lse[static_cast<long long>(b) * s.Hq + g * s.G + tid] = 0.f;
        return;
    }
    select_pair(a, pair, first_local_chunk(seq, s.W), sh, sel_dyn, nt >> 5);
    STAMP_MAX(3);
    pdl_launch_dependents();
}

// ------------------------------------------------------------------------------------------ attend
struct AttendSmem {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    int item_chunk[kMaxItems];     // chunk id, or -1 for an empty slot
    int item_row[kMaxItems];       // first row of the chunk in the K / V tensor maps
    uint8_t item_nvalid[kMaxItems];// valid rows (64, or fewer for the partial local chunk)
    float red[kConsumerWarps][8 * kD];
    int flag;
    int dead;                      // a bounded wait ran out: every consumer warp leaves at the next barrier
};

// first CTA whose item range [cta*N/n_ctas, (cta+1)*N/n_ctas) holds item x
__device__ inline int cta_of_item(long long x, long long N, int n_ctas) {
    return static_cast<int>(((x + 1) * n_ctas + N - 1) / N - 1);
}

__global__ void __launch_bounds__(kAttendThreads, 1)
decode_attend_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                     const DArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    AttendSmem& sm = *reinterpret_cast<AttendSmem*>(ring + kStages * kStageBytes);
    const Shape& s = a.s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int K = s.K, G = s.G, NL = max_local_slots(s.W), slots = K + NL;
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
    STAMP_MIN(6);
    pdl_wait();                                   // selection, weights and counters are visible
    STAMP_MIN(8);
    for (int j = tid; j < nitems; j += kAttendThreads) {
        const long long idx = lo + j;
        const int pair = static_cast<int>(idx / slots), slot = static_cast<int>(idx % slots);
        const int n = a.pair_n[pair];
        int c = -1, nv = kS;
        if (n >= 0) {
            if (slot < K) {
                c = slot < n ? a.sel[static_cast<long long>(pair) * K + slot] : -1;
            } else {
                // slot K + r: chunk lc + r of the local window; only the query's own chunk can be partial
                const int seq = query_seq_len(a, pair / s.Hkv);
                const int ci = (seq - 1) / kS;
                c = first_local_chunk(seq, s.W) + (slot - K);
                if (c > ci) c = -1;
                else if (c == ci) nv = (seq - 1) % kS + 1;
            }
        }
        int row = 0;
        if (c >= 0) {
            if (a.block_table) {
                const int page = a.block_table[static_cast<long long>(pair / s.Hkv / s.qps) * s.C + c];
                if (page < 0 || page >= a.num_pages) {       // flag it and skip the chunk
                    set_status(a.status, kDevBadIndex);
                    c = -1;
                } else {
                    row = (page * s.Hkv + pair % s.Hkv) * kS;
                }
            } else {
                row = ((pair / s.Hkv / s.qps) * s.Hkv + pair % s.Hkv) * s.T + c * kS;
            }
        }
        sm.item_chunk[j] = c;
        sm.item_row[j] = row;
        sm.item_nvalid[j] = static_cast<uint8_t>(nv);
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
                const int row = sm.item_row[j];
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
                        float* dst = a.loc_o + ((static_cast<long long>(pair) * NL + (slot - K)) * G + gq) * kD;
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            *reinterpret_cast<float2*>(dst + i * 8 + 2 * t) = make_float2(ol[i][0], ol[i][1]);
                        if (t == 0) a.loc_lam[(pair * NL + (slot - K)) * G + gq] = m * s.scale + __logf(z);
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
                {
                float acc = 0.f;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) acc += sm.red[w][x];      // fixed order: deterministic
                dst[x] = acc;
            }
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
            const int seq_b = query_seq_len(a, b);
            const int nl = (seq_b - 1) / kS - first_local_chunk(seq_b, s.W) + 1;
            for (int x = tid; x < G * kD; x += kConsumerWarps * 32) {
                const int h = x / kD;
                float A = 0.f;
                const float* src = a.part + static_cast<long long>(pair) * a.max_parts * G * kD + x;
                for (int pidx = 0; pidx < nparts; ++pidx) A += __ldcg(src + static_cast<long long>(pidx) * G * kD);
                // selected part first, then the chunks of the local window (masses lam_r, outputs o_r) folded in
                // one at a time with a running maximum (fixed order: deterministic)
                float Mx = -INFINITY, den = 0.f, num = 0.f;
                if (n_sel > 0) {
                    Mx = a.Rh[pair * G + h];
                    den = a.Eh[pair * G + h];
                    num = A;
                }
                const float* lam_p = a.loc_lam + pair * NL * G + h;
                const float* o_p = a.loc_o + static_cast<long long>(pair) * NL * G * kD + x;
#pragma unroll 2
                for (int r = 0; r < nl; ++r) {
                    const float lam = __ldcg(lam_p + r * G);
                    const float ol = __ldcg(o_p + static_cast<long long>(r) * G * kD);
                    const float nm = fmaxf(Mx, lam);
                    const float f = __expf(Mx - nm), wl = __expf(lam - nm);
                    den = fmaf(den, f, wl);
                    num = fmaf(num, f, wl * ol);
                    Mx = nm;
                }
                const float res = num / den;
                const float lse = Mx + __logf(den);
                const long long orow = static_cast<long long>(b) * s.Hq + g * G + h;
                a.out[orow * kD + (x % kD)] = __float2bfloat16_rn(res);
                if ((x % kD) == 0) a.lse[orow] = lse;
            }
        }
        asm volatile("bar.sync 1, %0;" ::"r"(kConsumerWarps * 32));
        j0 = j1;
        if (dead) break;
    }
    STAMP_MAX(7);
}

// HILS_DECODE_SCORE=segments keeps the scoring kernel with one CTA per 256-chunk segment even where the streaming one
// applies (for tuning runs and to cross-check the two).
const bool g_score_per_segment = [] {
    const char* e = getenv("HILS_DECODE_SCORE");
    return e != nullptr && e[0] == 's';
}();

struct Plan {
    int n_ctas, max_parts, Cpad;
    size_t off_u, off_uh, off_wgt, off_R, off_E, off_n, off_done, off_part, off_loco, off_loclam, total;
};

// The streaming scoring kernel (and with it the table of per-head scores) applies to one landmark row per KV head.
bool score_streams(const Shape& s) {
    return s.Hl == s.Hkv && static_cast<long long>(s.B) * s.Hkv <= kScMaxPairs && !g_score_per_segment;
}

Plan make_plan(const Shape& s, int n_sm) {
    Plan p;
    const long long pairs = static_cast<long long>(s.B) * s.Hkv;
    const int slots = s.K + max_local_slots(s.W);
    const long long N = pairs * slots;
    long long ctas = n_sm;
    if ((N + ctas - 1) / ctas + 1 > kMaxItems) ctas = (N + kMaxItems - 2) / (kMaxItems - 1);
    if (ctas > N) ctas = N;
    p.n_ctas = static_cast<int>(ctas);
    const long long per = N / ctas;                               // every CTA gets per or per+1 items
    p.max_parts = static_cast<int>((slots + per - 1) / per) + 1;
    if (p.max_parts > slots) p.max_parts = slots;
    p.Cpad = (s.C + 63) / 64 * 64;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = (off + bytes + 255) / 256 * 256; return o; };
    p.off_u = take(sizeof(float) * pairs * p.Cpad);
    p.off_uh = take(score_streams(s) ? sizeof(float) * pairs * s.G * p.Cpad : 0);
    p.off_wgt = take(sizeof(float) * pairs * s.G * s.K);
    p.off_R = take(sizeof(float) * pairs * s.G);
    p.off_E = take(sizeof(float) * pairs * s.G);
    p.off_n = take(sizeof(int) * pairs);
    p.off_done = take(sizeof(int) * pairs);
    p.off_part = take(sizeof(float) * pairs * p.max_parts * s.G * kD);
    p.off_loco = take(sizeof(float) * pairs * max_local_slots(s.W) * s.G * kD);
    p.off_loclam = take(sizeof(float) * pairs * max_local_slots(s.W) * s.G);
    p.total = off;
    return p;
}

}  // namespace

bool decode_fast_supports(const Shape& s, int dtype) {
    return dtype == HILS_BF16 && s.is_decode && s.d == kD && s.S == kS && s.W >= 1 && max_local_slots(s.W) <= 16 && (s.Hl == s.Hkv || s.Hl == s.Hq) && s.G <= 8 &&
           s.K >= 1 && s.K <= 128 && static_cast<long long>(s.B) * s.Hkv * s.T < (1ll << 31) &&
           static_cast<long long>(s.B) * s.Hkv <= 65535 && s.C < (1 << 24);
}

size_t decode_fast_scratch_bytes(const Shape& s) {
    // sized for the largest CTA count the launcher may use, independent of the device queried at run time
    // the larger of the layouts for this device's SM count, a B200's 148 and a single CTA
    size_t n = make_plan(s, 148).total;
    const size_t n1 = make_plan(s, 1).total, nd = make_plan(s, sm_count()).total;
    n = n1 > n ? n1 : n;
    return nd > n ? nd : n;
}

int launch_decode_fast(const Shape& s, const Tensors& t, cudaStream_t stream) {
    const Plan p = make_plan(s, sm_count());
    if (t.scratch_bytes < p.total) return HILS_ERR_WORKSPACE;
    const int pairs = s.B * s.Hkv;
    char* sc = static_cast<char*>(t.scratch);
    DArgs a;
    a.s = s;
    a.q = static_cast<const __nv_bfloat16*>(t.q);
    a.q_route = static_cast<const __nv_bfloat16*>(t.q_route ? t.q_route : t.q);
    a.lm = static_cast<const __nv_bfloat16*>(t.landmarks);
    a.bias = t.bias;
    a.seq_lens = t.seq_lens;
    a.out = static_cast<__nv_bfloat16*>(t.out);
    a.lse = t.lse;
    a.sel = t.sel_idx;
    a.status = t.status;
    a.u = reinterpret_cast<float*>(sc + p.off_u);
    a.uh = score_streams(s) ? reinterpret_cast<float*>(sc + p.off_uh) : nullptr;
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
    a.block_table = t.block_table;
    a.num_pages = t.num_pages;

    CUtensorMap map_k, map_v;
    const uint64_t rows = t.block_table ? static_cast<uint64_t>(t.num_pages) * s.Hkv * kS
                                        : static_cast<uint64_t>(pairs / s.qps) * s.T;
    if (!make_bf16_2d_map(&map_k, t.k, rows, kD, 64, kS) || !make_bf16_2d_map(&map_v, t.v, rows, kD, 64, kS))
        return HILS_ERR_CUDA;

    const size_t attend_smem = kStages * kStageBytes + sizeof(AttendSmem) + 1024;
    static PerDeviceOnce attr_once;
    if (attr_once.pending()) {
        if (cudaFuncSetAttribute(decode_attend_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(attend_smem)) != cudaSuccess ||
            cudaFuncSetAttribute(decode_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(sel_dyn_bytes(kSelMaxWarps, kSelKeyCap))) != cudaSuccess)
            return HILS_ERR_CUDA;
        attr_once.done();
    }

    if (score_streams(s)) {
        CUtensorMap map_lm;
        if (!make_bf16_2d_map(&map_lm, t.landmarks, static_cast<uint64_t>(s.B / s.qps) * s.Hl * s.C, kD, 64, kS))
            return HILS_ERR_CUDA;
        const size_t sc_smem = kScStages * kScStageBytes + sizeof(ScoreSmem) + 1024;
        static PerDeviceOnce sc_once;
        if (sc_once.pending()) {
            if (cudaFuncSetAttribute(decode_score_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     static_cast<int>(sc_smem)) != cudaSuccess)
                return HILS_ERR_CUDA;
            sc_once.done();
        }
        decode_score_stream_kernel<<<sm_count(), kScThreads, sc_smem, stream>>>(map_lm, a);
    } else {
        const int nseg = (s.C + kScoreChunksPerCta - 1) / kScoreChunksPerCta;
        decode_score_kernel<<<dim3(nseg > 0 ? nseg : 1, pairs), kScoreThreads, 0, stream>>>(a);
    }
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
    cfg.dynamicSmemBytes = 0;
    {
        const int cmax = (s.T - 1) / kS;                       // candidates of the longest possible sequence
        const int nw = cmax <= 1024 ? 4 : (cmax <= 4096 ? 8 : kSelMaxWarps);
        const size_t need = sel_dyn_bytes(nw, cmax < kSelKeyCap ? cmax : 0);
        cfg.blockDim = dim3(nw * 32);
        cfg.dynamicSmemBytes = need;
        if (cudaLaunchKernelEx(&cfg, decode_select_kernel, a) != cudaSuccess) return HILS_ERR_CUDA;
    }
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
// library image: every GPU that loads libhils.so carries these 16 MiB until the process exits.
constexpr size_t kNoAllocBytes = 16u << 20;
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
    // (No lock around this cache: two host threads that make a device's first call at the same moment both look the
    // address up and both store the same value.)
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
