// Backward of the HiLS operator through `out` with the selection held fixed: the chain rule applied to
// Eq. (HiLS weights) / App. C (the paper states only that the loss reaches the landmarks through these
// weights, Sec. 3.2).  With w_tj the final weight of key j of slot t, g_t = dout . o_t, D = dout . out:
//     selected chunk c:  w_j = alpha_c p_j,   d s_j = w_j (dout . v_j - g_c),   d lambda_c = alpha_c (g_c - D)
//                        alpha_c = exp(s^h_c - lse),  s^h_c = scale q . k'_c + b'_c
//     local span:        w_j = exp(s_j - lse),        d s_j = w_j (dout . v_j - D)
//     d v_j += w_j dout,   d q += scale d s_j k_j,   d k_j += scale d s_j q,
//     d q += scale d lambda_c k'_c,   d k'_c += scale d lambda_c q,   d b'_c += d lambda_c.
//
// This file: the shape-agnostic kernel on CUDA cores (fp32 and bf16, any head dim that is a multiple of 32,
// any chunk size, window and landmark-head layout): one warp per (sequence, query head, query row); d q is
// owned by the warp, the other four gradients are accumulated with fp32 atomics.
#include "internal.h"

namespace hils {
namespace {

constexpr int kBwdWarps = 4;

struct BArgs {
    Shape s;
    const void* q;
    const void* k;
    const void* v;
    const void* lm;
    const float* bias;
    const void* out;
    const float* lse;
    const int32_t* sel;
    const void* dout;
    float* dq;
    float* dk;
    float* dv;
    float* dlm;
    float* dbias;
    int* status;
};

// One pass over keys [lo, hi) of a slot, a block of 32 keys at a time (lane = key): logits s_j and
// t_j = dout . v_j.  MODE 0 accumulates the slot's softmax statistics (m, Z, sum_j e^{s_j - m} t_j); MODE 1 turns
// them into d s_j and w_j and applies the three updates.  `shift` is what the exponent is taken against
// (the slot's own m + log Z - log alpha for a selected chunk, lse for the local span) and `sub` is g_c or D.
template <typename T, int NE, int MODE>
__device__ inline void span_pass(const BArgs& a, const float* sq, const float* sdo, const T* kbase, const T* vbase,
                                 float* dkbase, float* dvbase, int lo, int hi, int lane, float& m, float& Z,
                                 float& gt, float shift, float sub, float (&dq)[NE]) {
    const int d = a.s.d;
    const float scale = a.s.scale;
    for (int base = lo; base < hi; base += 32) {
        const int j = base + lane;
        float sc = -INFINITY, tj = 0.f;
        if (j < hi) {
            const T* krow = kbase + static_cast<long long>(j) * d;
            const T* vrow = vbase + static_cast<long long>(j) * d;
            float a0 = 0.f, a1 = 0.f;
            for (int t = 0; t < d; t += 8) {
                float x[8], y[8];
                load8(krow + t, x);
                load8(vrow + t, y);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    a0 = fmaf(x[e], sq[t + e], a0);
                    a1 = fmaf(y[e], sdo[t + e], a1);
                }
            }
            sc = a0 * scale;
            tj = a1;
        }
        if (MODE == 0) {
            const float mn = fmaxf(m, warp_max(sc));
            const float corr = __expf(m - mn);
            const float e = (j < hi) ? __expf(sc - mn) : 0.f;
            Z = Z * corr + warp_sum(e);
            gt = gt * corr + warp_sum(e * tj);
            m = mn;
        } else {
            const float w = (j < hi) ? __expf(sc - shift) : 0.f;
            const float ds = w * (tj - sub) * scale;
            const int cnt = min(32, hi - base);
            for (int jj = 0; jj < cnt; ++jj) {
                const float dsj = __shfl_sync(kFullMask, ds, jj);
                const float wj = __shfl_sync(kFullMask, w, jj);
                const long long row = static_cast<long long>(base + jj) * d;
#pragma unroll
                for (int e = 0; e < NE; ++e) {
                    const int x = e * 32 + lane;
                    if (e * 32 < d) {
                        dq[e] = fmaf(dsj, to_f32(kbase[row + x]), dq[e]);
                        atomicAdd(dkbase + row + x, dsj * sq[x]);
                        atomicAdd(dvbase + row + x, wj * sdo[x]);
                    }
                }
            }
        }
    }
}

template <typename T, int NE>
__global__ void __launch_bounds__(kBwdWarps * 32) generic_backward_kernel(const BArgs a) {
    extern __shared__ float bsm[];
    const Shape& s = a.s;
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const long long w = static_cast<long long>(blockIdx.x) * kBwdWarps + wib;
    const long long total = static_cast<long long>(s.B) * s.Hq * s.R;
    if (w >= total) return;
    const int r = static_cast<int>(w % s.R);
    const int h = static_cast<int>((w / s.R) % s.Hq);
    const int b = static_cast<int>(w / (static_cast<long long>(s.R) * s.Hq));
    const int g = h / s.G, d = s.d;
    const long long orow = (static_cast<long long>(b) * s.Hq + h) * s.R + r;
    const int pos = s.pos0 + r;
    const int lo = local_lo(pos, s.W, s.S);
    const int ncand = lo / s.S;

    float* sq = bsm + static_cast<size_t>(wib) * 2 * d;
    float* sdo = sq + d;
    const T* q = static_cast<const T*>(a.q) + orow * d;
    const T* dout = static_cast<const T*>(a.dout) + orow * d;
    const T* out = static_cast<const T*>(a.out) + orow * d;
    float dd = 0.f;
    for (int t = lane; t < d; t += 32) {
        sq[t] = to_f32(q[t]);
        sdo[t] = to_f32(dout[t]);
        dd = fmaf(sdo[t], to_f32(out[t]), dd);
    }
    const float D = warp_sum(dd);                       // dout . out
    const float lse = a.lse[orow];
    __syncwarp();

    const long long kvoff = (static_cast<long long>(b) * s.Hkv + g) * s.T * d;
    const T* kg = static_cast<const T*>(a.k) + kvoff;
    const T* vg = static_cast<const T*>(a.v) + kvoff;
    float* dkg = a.dk + kvoff;
    float* dvg = a.dv + kvoff;
    const int hl = (s.Hl == s.Hq) ? h : g;
    const long long lmoff = (static_cast<long long>(b) * s.Hl + hl) * s.C;
    const T* lm = static_cast<const T*>(a.lm) + lmoff * d;
    const float* bias = a.bias ? a.bias + lmoff : nullptr;
    const int32_t* sel = a.sel + ((static_cast<long long>(b) * s.Hkv + g) * s.R + r) * s.K;

    float dq[NE];
#pragma unroll
    for (int e = 0; e < NE; ++e) dq[e] = 0.f;
    float m, Z, gt;

    // the local span: its keys' final weights are exp(s_j - lse) and its mass is their own log-sum-exp
    span_pass<T, NE, 1>(a, sq, sdo, kg, vg, dkg, dvg, lo, pos + 1, lane, m, Z, gt, lse, D, dq);

    for (int t = 0; t < s.K; ++t) {
        const int c = sel[t];
        if (c < 0) continue;
        if (c >= ncand) {
            if (lane == 0) set_status(a.status, kDevBadIndex);
            continue;
        }
        float dotp = 0.f;
        for (int x = lane; x < d; x += 32) dotp = fmaf(sq[x], to_f32(lm[static_cast<long long>(c) * d + x]), dotp);
        float lam = warp_sum(dotp) * s.scale;
        if (bias) lam += bias[c];
        m = -INFINITY;
        Z = 0.f;
        gt = 0.f;
        span_pass<T, NE, 0>(a, sq, sdo, kg, vg, dkg, dvg, c * s.S, (c + 1) * s.S, lane, m, Z, gt, 0.f, 0.f, dq);
        const float gc = gt / Z;                         // dout . o_c
        const float alpha = __expf(lam - lse);
        const float dlam = alpha * (gc - D);
        // w_j = alpha e^{s_j - m} / Z = exp(s_j - (m + log Z - (lam - lse)))
        span_pass<T, NE, 1>(a, sq, sdo, kg, vg, dkg, dvg, c * s.S, (c + 1) * s.S, lane, m, Z, gt,
                            m + __logf(Z) - (lam - lse), gc, dq);
        const float sdl = s.scale * dlam;
        float* dlm = a.dlm + (lmoff + c) * d;
#pragma unroll
        for (int e = 0; e < NE; ++e) {
            const int x = e * 32 + lane;
            if (e * 32 < d) {
                dq[e] = fmaf(sdl, to_f32(lm[static_cast<long long>(c) * d + x]), dq[e]);
                atomicAdd(dlm + x, sdl * sq[x]);
            }
        }
        if (lane == 0 && a.dbias) atomicAdd(a.dbias + lmoff + c, dlam);
    }
#pragma unroll
    for (int e = 0; e < NE; ++e)
        if (e * 32 < d) a.dq[orow * d + e * 32 + lane] = dq[e];
}

template <typename T>
int launch_bwd_typed(const BArgs& a, cudaStream_t stream) {
    const Shape& s = a.s;
    const long long warps = static_cast<long long>(s.B) * s.Hq * s.R;
    const unsigned blocks = static_cast<unsigned>((warps + kBwdWarps - 1) / kBwdWarps);
    const size_t smem = sizeof(float) * kBwdWarps * 2 * s.d;
    const int ne = s.d / 32;
    if (ne <= 2) generic_backward_kernel<T, 2><<<blocks, kBwdWarps * 32, smem, stream>>>(a);
    else if (ne <= 4) generic_backward_kernel<T, 4><<<blocks, kBwdWarps * 32, smem, stream>>>(a);
    else generic_backward_kernel<T, 8><<<blocks, kBwdWarps * 32, smem, stream>>>(a);
    if (cudaGetLastError() != cudaSuccess) return HILS_ERR_CUDA;
    trace_mark("generic_backward", stream);
    return 1;
}

}  // namespace

int launch_backward_generic(const Shape& s, int dtype, const BackwardTensors& t, cudaStream_t stream) {
    if (!generic_supports(s)) return HILS_ERR_UNSUPPORTED;
    BArgs a{s, t.q, t.k, t.v, t.landmarks, t.bias, t.out, t.lse, t.sel_idx, t.dout,
            t.dq, t.dk, t.dv, t.dlandmarks, t.dbias, t.status};
    if (dtype == HILS_F32) return launch_bwd_typed<float>(a, stream);
    return launch_bwd_typed<__nv_bfloat16>(a, stream);
}

}  // namespace hils
