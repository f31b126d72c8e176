// Shape-agnostic HiLS kernels on CUDA cores: one warp per (sequence, KV group, query row) for
// scoring + top-K selection, one warp per (sequence, query head, query row) for attention.
// They cover fp32 and bf16, any head dim that is a multiple of 32 (<= 256), any chunk size and
// any local window, prefill and decode.  They are the correctness anchor and the fall-back for
// shapes the tensor-core / bandwidth-tuned kernels do not take.
#include "internal.h"

namespace hils {
namespace {

constexpr int kWarpsPerBlock = 4;

struct GArgs {
    Shape s;
    const void* q;
    const void* q_route;   // routing query for the surrogate scores (= q unless a separate one was given)
    const void* k;
    const void* v;
    const void* lm;
    const float* bias;
    const int32_t* seq_lens;
    void* out;
    float* lse;
    int32_t* sel;
    int* status;
};

// Position of query row r of sequence b, or -1 if the decode length is invalid.
__device__ inline int row_position(const GArgs& a, int b, int r) {
    if (!a.s.is_decode) return a.s.pos0 + r;
    const int n = a.seq_lens[b];
    if (n < 1 || n > a.s.T) return -1;
    return n - 1;
}

// Insert key x into the descending list held as lst[j] of lane l <-> index j*32+l, keeping K entries.
template <int NR>
__device__ inline void list_insert(unsigned long long (&lst)[NR], unsigned long long x, int K, int lane) {
    int pos = 0;
#pragma unroll
    for (int j = 0; j < NR; ++j) pos += __popc(__ballot_sync(kFullMask, lst[j] > x));
#pragma unroll
    for (int j = NR - 1; j >= 0; --j) {
        const int idx = j * 32 + lane;
        unsigned long long up = __shfl_up_sync(kFullMask, lst[j], 1);
        unsigned long long carry = 0ull;
        if (j > 0) carry = __shfl_sync(kFullMask, lst[j - 1], 31);
        if (lane == 0) up = carry;
        unsigned long long nv = idx < pos ? lst[j] : (idx == pos ? x : up);
        if (idx >= K) nv = 0ull;
        lst[j] = nv;
    }
}

// Scoring (Eq. surrogate top-k, per head), group max (App. C) and exact top-K with ties to the
// lower chunk id.  One warp per (b, g, r); lane l scores chunk base+l.
template <typename T, int NR>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
generic_select_kernel(const GArgs a) {
    extern __shared__ float smem[];
    const Shape& s = a.s;
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const long long w = static_cast<long long>(blockIdx.x) * kWarpsPerBlock + wib;
    const long long total = static_cast<long long>(s.B) * s.Hkv * s.R;
    if (w >= total) return;
    const int r = static_cast<int>(w % s.R);
    const int g = static_cast<int>((w / s.R) % s.Hkv);
    const int b = static_cast<int>(w / (static_cast<long long>(s.R) * s.Hkv));
    int32_t* sel = a.sel + ((static_cast<long long>(b) * s.Hkv + g) * s.R + r) * s.K;
    const int pos = row_position(a, b, r);
    if (pos < 0) {
        if (lane == 0) set_status(a.status, kDevBadIndex);
        for (int t = lane; t < s.K; t += 32) sel[t] = -1;
        return;
    }
    const int ncand = local_lo(pos, s.W, s.S) / s.S;
    const int d = s.d, G = s.G;
    float* sq = smem + static_cast<size_t>(wib) * G * d;        // [G][d] queries of the group
    const T* q = static_cast<const T*>(a.q_route);       // selection scores use the routing query
    for (int x = lane; x < G * d; x += 32) {
        const int rr = x / d, t = x % d;
        sq[x] = to_f32(q[((static_cast<long long>(b) * s.Hq + g * G + rr) * s.R + r) * d + t]);
    }
    __syncwarp();

    unsigned long long lst[NR];
#pragma unroll
    for (int j = 0; j < NR; ++j) lst[j] = 0ull;
    unsigned long long thr = 0ull;
    const T* lm = static_cast<const T*>(a.lm);

    for (int base = 0; base < ncand; base += 32) {
        const int c = base + lane;
        unsigned long long key = 0ull;
        if (c < ncand) {
            float u = -INFINITY;
            for (int rr = 0; rr < G; ++rr) {
                const int hl = (s.Hl == s.Hq) ? (g * G + rr) : g;
                const T* row = lm + ((static_cast<long long>(b) * s.Hl + hl) * s.C + c) * d;
                const float* qv = sq + rr * d;
                float acc = 0.f;
                for (int t = 0; t < d; t += 8) {
                    float x[8];
                    load8(row + t, x);
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc = fmaf(x[e], qv[t + e], acc);
                }
                float sc = acc * s.scale;
                if (a.bias) sc += a.bias[(static_cast<long long>(b) * s.Hl + hl) * s.C + c];
                u = fmaxf(u, sc);
            }
            key = select_key(u, c);
        }
        unsigned pass = __ballot_sync(kFullMask, key > thr);
        while (pass) {
            const int src = __ffs(pass) - 1;
            pass &= pass - 1;
            const unsigned long long x = __shfl_sync(kFullMask, key, src);
            if (x > thr) {
                list_insert<NR>(lst, x, s.K, lane);
                thr = __shfl_sync(kFullMask, lst[(s.K - 1) >> 5], (s.K - 1) & 31);
            }
        }
    }

    // emit ascending chunk ids: rank of an id = number of selected ids below it
    const int n = ncand < s.K ? ncand : s.K;
#pragma unroll
    for (int j = 0; j < NR; ++j) {
        const int idx = j * 32 + lane;
        const int mine = (idx < n) ? key_chunk(lst[j]) : 0x7fffffff;
        int rank = 0;
#pragma unroll
        for (int j2 = 0; j2 < NR; ++j2) {
            for (int l = 0; l < 32; ++l) {
                const unsigned long long o = __shfl_sync(kFullMask, lst[j2], l);
                const int oi = (j2 * 32 + l < n) ? key_chunk(o) : 0x7fffffff;
                rank += (oi < mine) ? 1 : 0;
            }
        }
        if (idx < n) sel[rank] = mine;
    }
    for (int t = n + lane; t < s.K; t += 32) sel[t] = -1;
}

// Softmax attention of the warp's query (in shared memory) over rows [lo, hi) of one KV head,
// 32 keys at a time with a running max.  Returns m and Z; acc holds sum exp(s - m) * v.
// Lane l owns output elements e*32 + l.
template <typename T, int NE>
__device__ inline void attend_span(const float* sq, const T* kbase, const T* vbase, int lo, int hi, int d,
                                   float scale, int lane, float& m, float& Z, float (&acc)[NE]) {
    m = -INFINITY;
    Z = 0.f;
#pragma unroll
    for (int e = 0; e < NE; ++e) acc[e] = 0.f;
    for (int base = lo; base < hi; base += 32) {
        const int j = base + lane;
        float sc = -INFINITY;
        if (j < hi) {
            const T* row = kbase + static_cast<long long>(j) * d;
            float a0 = 0.f;
            for (int t = 0; t < d; t += 8) {
                float x[8];
                load8(row + t, x);
#pragma unroll
                for (int e = 0; e < 8; ++e) a0 = fmaf(x[e], sq[t + e], a0);
            }
            sc = a0 * scale;
        }
        const float mb = warp_max(sc);
        const float mn = fmaxf(m, mb);
        const float corr = __expf(m - mn);          // m = -inf on the first block -> 0
        const float p = (j < hi) ? __expf(sc - mn) : 0.f;
        Z = Z * corr + warp_sum(p);
#pragma unroll
        for (int e = 0; e < NE; ++e) acc[e] *= corr;
        const int cnt = min(32, hi - base);
        for (int jj = 0; jj < cnt; ++jj) {
            const float pj = __shfl_sync(kFullMask, p, jj);
            const T* vrow = vbase + static_cast<long long>(base + jj) * d;
#pragma unroll
            for (int e = 0; e < NE; ++e)
                if (e * 32 < d) acc[e] = fmaf(pj, to_f32(vrow[e * 32 + lane]), acc[e]);
        }
        m = mn;
    }
}

// Per-chunk attention, local attention and fusion (Eq. HiLS weights; App. C per-head weights).
// One warp per (b, h, r).
template <typename T, int NE>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
generic_attend_kernel(const GArgs a) {
    extern __shared__ float smem[];
    const Shape& s = a.s;
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const long long w = static_cast<long long>(blockIdx.x) * kWarpsPerBlock + wib;
    const long long total = static_cast<long long>(s.B) * s.Hq * s.R;
    if (w >= total) return;
    const int r = static_cast<int>(w % s.R);
    const int h = static_cast<int>((w / s.R) % s.Hq);
    const int b = static_cast<int>(w / (static_cast<long long>(s.R) * s.Hq));
    const int g = h / s.G, d = s.d;
    const long long orow = (static_cast<long long>(b) * s.Hq + h) * s.R + r;
    T* out = static_cast<T*>(a.out) + orow * d;
    const int pos = row_position(a, b, r);
    if (pos < 0) {
        for (int t = lane; t < d; t += 32) out[t] = from_f32<T>(0.f);
        if (lane == 0) a.lse[orow] = 0.f;
        return;
    }
    const int lo = local_lo(pos, s.W, s.S);
    const int ncand = lo / s.S;
    float* sq = smem + static_cast<size_t>(wib) * 2 * d;        // attention query, then routing query
    float* sr = sq + d;
    const T* q = static_cast<const T*>(a.q) + orow * d;
    const T* qr = static_cast<const T*>(a.q_route) + orow * d;
    for (int t = lane; t < d; t += 32) { sq[t] = to_f32(q[t]); sr[t] = to_f32(qr[t]); }
    __syncwarp();

    const T* kg = static_cast<const T*>(a.k) + (static_cast<long long>(b) * s.Hkv + g) * s.T * d;
    const T* vg = static_cast<const T*>(a.v) + (static_cast<long long>(b) * s.Hkv + g) * s.T * d;
    const int hl = (s.Hl == s.Hq) ? h : g;
    const T* lm = static_cast<const T*>(a.lm) + (static_cast<long long>(b) * s.Hl + hl) * s.C * d;
    const float* bias = a.bias ? a.bias + (static_cast<long long>(b) * s.Hl + hl) * s.C : nullptr;
    const int32_t* sel = a.sel + ((static_cast<long long>(b) * s.Hkv + g) * s.R + r) * s.K;

    // local branch first: lambda_loc = log Z_swa
    float m, Z, acc[NE], part[NE];
    attend_span<T, NE>(sq, kg, vg, lo, pos + 1, d, s.scale, lane, m, Z, part);
    float Mx = m + __logf(Z);
    float D = 1.f;
#pragma unroll
    for (int e = 0; e < NE; ++e) acc[e] = part[e] / Z;

    for (int t = 0; t < s.K; ++t) {
        const int c = sel[t];
        if (c < 0) continue;
        if (c >= ncand) {                       // never produced by the selection kernel
            if (lane == 0) set_status(a.status, kDevBadIndex);
            continue;
        }
        float dotp = 0.f;
        for (int x = lane; x < d; x += 32) dotp = fmaf(sr[x], to_f32(lm[static_cast<long long>(c) * d + x]), dotp);
        float lam = warp_sum(dotp) * s.scale;
        if (bias) lam += bias[c];
        attend_span<T, NE>(sq, kg, vg, c * s.S, (c + 1) * s.S, d, s.scale, lane, m, Z, part);
        const float Mn = fmaxf(Mx, lam);
        const float c_old = __expf(Mx - Mn), c_new = __expf(lam - Mn);
        D = D * c_old + c_new;
        const float wnew = c_new / Z;
#pragma unroll
        for (int e = 0; e < NE; ++e) acc[e] = acc[e] * c_old + part[e] * wnew;
        Mx = Mn;
    }
    const float inv = 1.f / D;
#pragma unroll
    for (int e = 0; e < NE; ++e)
        if (e * 32 < d) out[e * 32 + lane] = from_f32<T>(acc[e] * inv);
    if (lane == 0) a.lse[orow] = Mx + __logf(D);
}

template <typename T>
int launch_typed(const GArgs& a, cudaStream_t stream) {
    const Shape& s = a.s;
    const long long sel_warps = static_cast<long long>(s.B) * s.Hkv * s.R;
    const long long att_warps = static_cast<long long>(s.B) * s.Hq * s.R;
    const unsigned sel_blocks = static_cast<unsigned>((sel_warps + kWarpsPerBlock - 1) / kWarpsPerBlock);
    const unsigned att_blocks = static_cast<unsigned>((att_warps + kWarpsPerBlock - 1) / kWarpsPerBlock);
    const size_t sel_smem = sizeof(float) * kWarpsPerBlock * s.G * s.d;
    const size_t att_smem = sizeof(float) * kWarpsPerBlock * 2 * s.d;
    const int nr = (s.K + 31) / 32;
    if (nr <= 1) generic_select_kernel<T, 1><<<sel_blocks, kWarpsPerBlock * 32, sel_smem, stream>>>(a);
    else if (nr == 2) generic_select_kernel<T, 2><<<sel_blocks, kWarpsPerBlock * 32, sel_smem, stream>>>(a);
    else generic_select_kernel<T, 4><<<sel_blocks, kWarpsPerBlock * 32, sel_smem, stream>>>(a);
    if (cudaGetLastError() != cudaSuccess) return HILS_ERR_CUDA;
    trace_mark("generic_select", stream);
    const int ne = s.d / 32;
    if (ne <= 2) generic_attend_kernel<T, 2><<<att_blocks, kWarpsPerBlock * 32, att_smem, stream>>>(a);
    else if (ne <= 4) generic_attend_kernel<T, 4><<<att_blocks, kWarpsPerBlock * 32, att_smem, stream>>>(a);
    else generic_attend_kernel<T, 8><<<att_blocks, kWarpsPerBlock * 32, att_smem, stream>>>(a);
    if (cudaGetLastError() != cudaSuccess) return HILS_ERR_CUDA;
    trace_mark("generic_attend", stream);
    return 2;
}

}  // namespace

bool generic_supports(const Shape& s) {
    return s.d % 32 == 0 && s.d >= 32 && s.d <= 256 && s.K >= 1 && s.K <= 128 && s.G * s.d <= 2048 &&
           s.S >= 1;
}

int launch_generic(const Shape& s, int dtype, const Tensors& t, cudaStream_t stream) {
    if (!generic_supports(s)) return HILS_ERR_UNSUPPORTED;
    GArgs a{s, t.q, t.q_route ? t.q_route : t.q, t.k, t.v, t.landmarks, t.bias, t.seq_lens, t.out, t.lse, t.sel_idx, t.status};
    if (dtype == HILS_F32) return launch_typed<float>(a, stream);
    return launch_typed<__nv_bfloat16>(a, stream);
}

}  // namespace hils
