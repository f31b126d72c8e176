// Chunk summaries (Proposition 3.1, Eq. prop_q_c): k'_c = Attn(q'_c, K_c, K_c) and b'_c = entropy of the
// attention distribution of the chunk's learnable query over the chunk's keys.
//
// One warp per (sequence, landmark head, chunk).  The warp copies the chunk's keys into its own padded
// shared-memory tile with cp.async (every key byte is read from memory exactly once, 16 bytes per lane,
// coalesced), then
//   scores      lane l owns key rows l, l + 32, ...: a full dot product per row from shared memory (rows are
//               272-byte apart for d = 128 bf16, so a quarter warp touches all 32 banks once), no shuffles;
//   softmax     two warp reductions; b' = log Z - sum p (s - max);
//   k'          lane l owns d/32 output dimensions and runs over the rows.
// The loops are rolled (a first, fully unrolled register version was bound by instruction fetch at 20 % of
// the memory bandwidth).  The kernel is bound by HBM: algorithmic bytes = the keys of the summarised chunks.
#include "internal.h"

namespace hils {
namespace {

constexpr int kMaxS = 128;
constexpr int kMaxWarps = 4;

struct LArgs {
    int B, Hkv, Hl, C, S;
    long long T;
    float scale;
    const void* lq;
    const void* k;
    const int32_t* seq;
    void* lm;
    float* bias;
    int c0, cn;
};

__device__ __forceinline__ float elem_f32(float x) { return x; }
__device__ __forceinline__ float elem_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void elem_set(float& dst, float x) { dst = x; }
__device__ __forceinline__ void elem_set(__nv_bfloat16& dst, float x) { dst = __float2bfloat16_rn(x); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

// D = head dimension (32, 64, 128, 256).  Shared memory per warp: S rows of D * sizeof(T) + 16 bytes, D floats
// for the scaled query and kMaxS floats for the probabilities.
template <typename T, int D>
__global__ void landmark_summary_kernel(const LArgs a) {
    extern __shared__ __align__(16) uint8_t lsm[];
    constexpr int RB = D * static_cast<int>(sizeof(T));       // bytes per key row
    constexpr int RS = RB + 16;                               // row stride in shared memory
    constexpr int EPP = 16 / static_cast<int>(sizeof(T));     // elements per 16-byte piece
    constexpr int VPL = D / 32;                               // output dimensions per lane
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const size_t per_warp = static_cast<size_t>(a.S) * RS + D * sizeof(float) + kMaxS * sizeof(float);
    uint8_t* tile = lsm + warp * per_warp;
    float* qs = reinterpret_cast<float*>(tile + static_cast<size_t>(a.S) * RS);
    float* ps = qs + D;
    const long long item = static_cast<long long>(blockIdx.x) * nwarps + warp;
    const long long total = static_cast<long long>(a.B) * a.Hl * a.cn;
    if (item >= total) return;
    const int c = a.c0 + static_cast<int>(item % a.cn);
    const int hl = static_cast<int>((item / a.cn) % a.Hl);
    const int b = static_cast<int>(item / (static_cast<long long>(a.cn) * a.Hl));
    const int hkv = hl / (a.Hl / a.Hkv);
    long long len = a.seq ? a.seq[b] : a.T;
    len = len < 0 ? 0 : (len > a.T ? a.T : len);
    const long long j0 = static_cast<long long>(c) * a.S;
    const int n = static_cast<int>(len - j0 < 0 ? 0 : (len - j0 > a.S ? a.S : len - j0));
    const long long orow = (static_cast<long long>(b) * a.Hl + hl) * a.C + c;
    T* out = static_cast<T*>(a.lm) + orow * D + lane * VPL;
    if (n == 0) {
#pragma unroll
        for (int i = 0; i < VPL; ++i) elem_set(out[i], 0.f);
        if (lane == 0) a.bias[orow] = 0.f;
        return;
    }
    // ---- the chunk's keys -> shared memory (asynchronously), the scaled query meanwhile
    {
        const uint8_t* src = reinterpret_cast<const uint8_t*>(
            static_cast<const T*>(a.k) + ((static_cast<long long>(b) * a.Hkv + hkv) * a.T + j0) * D);
        constexpr int PPR = RB / 16;
        const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(tile));
        for (int x = lane; x < n * PPR; x += 32) {
            const int row = x / PPR, pc = x % PPR;
            cp_async16(dst + row * RS + pc * 16, src + static_cast<size_t>(row) * RB + pc * 16);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        const T* q = static_cast<const T*>(a.lq) + orow * D;
        for (int e = lane; e < D; e += 32) qs[e] = elem_f32(q[e]) * a.scale;
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncwarp();
    }
    // ---- scores s_j = scale * q'_c . k_j for the rows of this lane (slot r: row lane + 32 r)
    float sreg[kMaxS / 32];
#pragma unroll
    for (int r = 0; r < kMaxS / 32; ++r) {
        sreg[r] = -INFINITY;
        const int j = lane + 32 * r;
        if (j < n) {
            const uint8_t* row = tile + static_cast<size_t>(j) * RS;
            float s = 0.f;
#pragma unroll 4
            for (int pc = 0; pc < RB / 16; ++pc) {
                const uint4 raw = *reinterpret_cast<const uint4*>(row + pc * 16);
                const T* e = reinterpret_cast<const T*>(&raw);
#pragma unroll
                for (int i = 0; i < EPP; ++i) s = fmaf(qs[pc * EPP + i], elem_f32(e[i]), s);
            }
            sreg[r] = s;
        }
    }
    // ---- p = softmax(s), b' = -sum p log p = log Z - sum p (s - m)
    float m = -INFINITY;
#pragma unroll
    for (int r = 0; r < kMaxS / 32; ++r) m = fmaxf(m, sreg[r]);
    m = warp_max(m);
    float z = 0.f, pe[kMaxS / 32];
#pragma unroll
    for (int r = 0; r < kMaxS / 32; ++r) {
        pe[r] = sreg[r] == -INFINITY ? 0.f : __expf(sreg[r] - m);
        z += pe[r];
    }
    z = warp_sum(z);
    const float zi = 1.f / z;
    float psum = 0.f;
#pragma unroll
    for (int r = 0; r < kMaxS / 32; ++r) {
        const float pj = pe[r] * zi;
        if (pj > 0.f) psum = fmaf(pj, sreg[r] - m, psum);
        if (lane + 32 * r < n) ps[lane + 32 * r] = pj;
    }
    psum = warp_sum(psum);
    __syncwarp();
    // ---- k' = sum_j p_j k_j: this lane's VPL output dimensions over all rows
    float acc[VPL];
#pragma unroll
    for (int i = 0; i < VPL; ++i) acc[i] = 0.f;
    const uint8_t* col = tile + lane * VPL * sizeof(T);
#pragma unroll 8
    for (int j = 0; j < n; ++j) {
        const float pj = ps[j];
        const T* e = reinterpret_cast<const T*>(col + static_cast<size_t>(j) * RS);
#pragma unroll
        for (int i = 0; i < VPL; ++i) acc[i] = fmaf(pj, elem_f32(e[i]), acc[i]);
    }
#pragma unroll
    for (int i = 0; i < VPL; ++i) elem_set(out[i], acc[i]);
    if (lane == 0) a.bias[orow] = __logf(z) - psum;
}

template <typename T, int D>
int launch_one(const LArgs& a, cudaStream_t stream) {
    const long long total = static_cast<long long>(a.B) * a.Hl * a.cn;
    if (total == 0) return 0;
    const size_t per_warp = static_cast<size_t>(a.S) * (D * sizeof(T) + 16) + D * sizeof(float) + kMaxS * sizeof(float);
    int nw = static_cast<int>(69632 / per_warp);            // three 68 KB blocks per SM
    nw = nw < 1 ? 1 : (nw > kMaxWarps ? kMaxWarps : nw);
    const size_t smem = per_warp * nw;
    if (smem > 227 * 1024) return HILS_ERR_UNSUPPORTED;
    static size_t attr_bytes = 0;                             // per instantiation
    if (smem > attr_bytes) {
        if (cudaFuncSetAttribute(landmark_summary_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem)) != cudaSuccess)
            return HILS_ERR_CUDA;
        attr_bytes = smem;
    }
    const long long blocks = (total + nw - 1) / nw;
    if (blocks > 0x7fffffffll) return HILS_ERR_UNSUPPORTED;
    landmark_summary_kernel<T, D><<<static_cast<unsigned>(blocks), nw * 32, smem, stream>>>(a);
    return cudaGetLastError() == cudaSuccess ? 1 : HILS_ERR_CUDA;
}

template <typename T>
int launch_typed(const LArgs& a, int d, cudaStream_t stream) {
    switch (d) {
        case 32: return launch_one<T, 32>(a, stream);
        case 64: return launch_one<T, 64>(a, stream);
        case 128: return launch_one<T, 128>(a, stream);
        case 256: return launch_one<T, 256>(a, stream);
        default: return HILS_ERR_UNSUPPORTED;
    }
}

}  // namespace

bool landmark_summary_supports(int d, int S) { return (d == 32 || d == 64 || d == 128 || d == 256) && S >= 1 && S <= kMaxS; }

int launch_landmark_summary(int dtype, int B, int Hkv, int Hl, int C, int d, int S, long long T, float scale,
                            const void* lq, const void* k, const int32_t* seq_lens, int c0, int cn, void* landmarks,
                            float* bias, cudaStream_t stream) {
    LArgs a{B, Hkv, Hl, C, S, T, scale, lq, k, seq_lens, landmarks, bias, c0, cn};
    return dtype == HILS_F32 ? launch_typed<float>(a, d, stream) : launch_typed<__nv_bfloat16>(a, d, stream);
}

}  // namespace hils
