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
#include "tma.cuh"

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

// ---- bf16, d = 128, S = 64, at most 8 landmark heads per KV head: both contractions on mma.sync ----
// One warp per (sequence, KV head, chunk): the chunk's keys arrive as two TMA boxes (128B swizzle) in the warp's
// own 16 KB tile; scores of all landmark heads of the KV head in one pass (the heads are the MMA rows), then
// k' = P K with P split into two bf16 terms (p = hi + lo), so that the weights keep 16 bits of mantissa.
constexpr int kTcWarps = 4;
constexpr int kTcTileBytes = 64 * 128 * 2;

struct TcSmemW {
    uint64_t bar;
};

__global__ void __launch_bounds__(kTcWarps * 32)
landmark_summary_tc_kernel(const __grid_constant__ CUtensorMap map_k, const LArgs a, int* timeout_flag) {
    extern __shared__ uint8_t lsm_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(lsm_raw) + 1023) & ~uintptr_t(1023));
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint8_t* tile = base + warp * kTcTileBytes;
    TcSmemW& sw = reinterpret_cast<TcSmemW*>(base + kTcWarps * kTcTileBytes)[warp];
    const int per = a.Hl / a.Hkv;                              // landmark heads per KV head (MMA rows), <= 8
    const long long item = static_cast<long long>(blockIdx.x) * kTcWarps + warp;
    const long long total = static_cast<long long>(a.B) * a.Hkv * a.cn;
    if (item >= total) return;
    const int c = a.c0 + static_cast<int>(item % a.cn);
    const int hkv = static_cast<int>((item / a.cn) % a.Hkv);
    const int b = static_cast<int>(item / (static_cast<long long>(a.cn) * a.Hkv));
    long long len = a.seq ? a.seq[b] : a.T;
    len = len < 0 ? 0 : (len > a.T ? a.T : len);
    const long long j0 = static_cast<long long>(c) * 64;
    const int n = static_cast<int>(len - j0 < 0 ? 0 : (len - j0 > 64 ? 64 : len - j0));
    const int gq = lane >> 2, t = lane & 3;
    const long long orow0 = (static_cast<long long>(b) * a.Hl + hkv * per) * a.C + c;      // head 0 of this KV head
    __nv_bfloat16* lm = static_cast<__nv_bfloat16*>(a.lm);
    if (n == 0) {
        for (int x = lane; x < per * 64; x += 32)
            *reinterpret_cast<uint32_t*>(lm + (orow0 + static_cast<long long>(x >> 6) * a.C) * 128 + (x & 63) * 2) = 0u;
        if (lane < per) a.bias[orow0 + static_cast<long long>(lane) * a.C] = 0.f;
        return;
    }
    if (lane == 0) {
        mbar_init(&sw.bar, 1);
        mbar_fence_init();
        const int row = static_cast<int>((static_cast<long long>(b) * a.Hkv + hkv) * a.T + j0);
        mbar_expect_tx(&sw.bar, kTcTileBytes);
        tma_load_2d(tile, &map_k, &sw.bar, 0, row);
        tma_load_2d(tile + 8192, &map_k, &sw.bar, 64, row);
    }
    // A operand: the `per` learnable queries of this KV head in rows 0..per-1 (loaded while the keys travel)
    uint32_t aq[8][2];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) { aq[ks][0] = 0u; aq[ks][1] = 0u; }
    if (gq < per) {
        const __nv_bfloat16* qrow = static_cast<const __nv_bfloat16*>(a.lq) + (orow0 + static_cast<long long>(gq) * a.C) * 128;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            aq[ks][0] = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 2 * t);
            aq[ks][1] = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8 + 2 * t);
        }
    }
    __syncwarp();
    if (!mbar_wait(&sw.bar, 0)) {
        // the bounded wait ran out (never seen: the copy has a valid map): mark the chunk's bias NaN and leave
        if (lane == 0 && timeout_flag) atomicExch(timeout_flag, 1);
        if (lane < per) a.bias[orow0 + static_cast<long long>(lane) * a.C] = __int_as_float(0x7fc00000);
        return;
    }
    if (n < 64) {
        // rows past the sequence end may hold anything: zero them before they meet probabilities of 0
        for (int x = lane; x < (64 - n) * 16; x += 32) {
            const int row = n + (x >> 4), piece = x & 15;
            *reinterpret_cast<uint4*>(tile + (piece >> 3) * 8192 + swz128(row, piece & 7)) = make_uint4(0u, 0u, 0u, 0u);
        }
        __syncwarp();
    }
    const uint32_t ks_addr = smem_u32(tile);
    float sc[8][4];
    qk_tile(aq, ks_addr, lane, sc);                             // sc[nt][0..1]: row gq, keys nt*8 + 2t, +1
    const float sl = a.scale;
    float m = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
        const int key = nt * 8 + 2 * t;
        sc[nt][0] = key < n ? sc[nt][0] * sl : -INFINITY;
        sc[nt][1] = key + 1 < n ? sc[nt][1] * sl : -INFINITY;
        m = fmaxf(m, fmaxf(sc[nt][0], sc[nt][1]));
    }
    m = fmaxf(m, __shfl_xor_sync(kFullMask, m, 1));
    m = fmaxf(m, __shfl_xor_sync(kFullMask, m, 2));
    float z = 0.f, ps = 0.f, e[8][2];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
        e[nt][0] = sc[nt][0] == -INFINITY ? 0.f : __expf(sc[nt][0] - m);
        e[nt][1] = sc[nt][1] == -INFINITY ? 0.f : __expf(sc[nt][1] - m);
        z += e[nt][0] + e[nt][1];
    }
    z += __shfl_xor_sync(kFullMask, z, 1);
    z += __shfl_xor_sync(kFullMask, z, 2);
    const float zi = 1.f / z;
    float phi[8][4], plo[8][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const float p = e[nt][x] * zi;
            if (p > 0.f) ps = fmaf(p, sc[nt][x] - m, ps);
            const float hi = __bfloat162float(__float2bfloat16_rn(p));
            phi[nt][x] = hi;
            plo[nt][x] = p - hi;
        }
        phi[nt][2] = phi[nt][3] = plo[nt][2] = plo[nt][3] = 0.f;
    }
    ps += __shfl_xor_sync(kFullMask, ps, 1);
    ps += __shfl_xor_sync(kFullMask, ps, 2);
    float o[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    pv_tile(phi, ks_addr, lane, o);                             // the keys are the "values" of Attn(q', K, K)
    pv_tile(plo, ks_addr, lane, o);
    if (gq < per) {
        __nv_bfloat16* dst = lm + (orow0 + static_cast<long long>(gq) * a.C) * 128;
#pragma unroll
        for (int i = 0; i < 16; ++i)
            *reinterpret_cast<uint32_t*>(dst + i * 8 + 2 * t) = pack_bf16(o[i][0], o[i][1]);
        if (t == 0) a.bias[orow0 + static_cast<long long>(gq) * a.C] = __logf(z) - ps;
    }
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
    static const bool no_tc = [] { const char* e = getenv("HILS_LANDMARK_NO_MMA"); return e && e[0] == '1'; }();
    const long long rows = static_cast<long long>(B) * Hkv * T;
    if (!no_tc && dtype == HILS_BF16 && d == 128 && S == 64 && Hl / Hkv <= 8 && rows < (1ll << 31)) {
        const long long total = static_cast<long long>(B) * Hkv * cn;
        if (total == 0) return 0;
        CUtensorMap map_k;
        if (!make_bf16_2d_map(&map_k, k, static_cast<uint64_t>(rows), 128, 64, 64)) return HILS_ERR_CUDA;
        const size_t smem = kTcWarps * kTcTileBytes + kTcWarps * sizeof(TcSmemW) + 1024;
        static PerDeviceOnce attr_once;
        if (attr_once.pending()) {
            if (cudaFuncSetAttribute(landmark_summary_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     static_cast<int>(smem)) != cudaSuccess)
                return HILS_ERR_CUDA;
            attr_once.done();
        }
        const long long blocks = (total + kTcWarps - 1) / kTcWarps;
        if (blocks > 0x7fffffffll) return HILS_ERR_UNSUPPORTED;
        landmark_summary_tc_kernel<<<static_cast<unsigned>(blocks), kTcWarps * 32, smem, stream>>>(map_k, a, nullptr);
        return cudaGetLastError() == cudaSuccess ? 1 : HILS_ERR_CUDA;
    }
    return dtype == HILS_F32 ? launch_typed<float>(a, d, stream) : launch_typed<__nv_bfloat16>(a, d, stream);
}

}  // namespace hils
