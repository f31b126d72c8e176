// Shared device/host helpers of the HiLS CUDA library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/hils.h"

namespace hils {

constexpr int kStatusBytes = 256;     // head of every workspace: device status word + padding
constexpr unsigned kFullMask = 0xffffffffu;

// Device status word values (first int32 of the workspace); 0 = ok.
constexpr int kDevTimeout = 1;
constexpr int kDevBadIndex = 2;

struct Shape {
    int B, Hq, Hkv, Hl, G;
    int R;          // query rows per sequence: L for prefill, 1 for decode
    int T;          // kv tokens allocated per (b, kv head)
    int C;          // landmark rows allocated per (b, landmark head)
    int d, S, K, W;
    float scale;
    int is_decode;
    int pos0;       // prefill: sequence position of query row 0 (rows are the tokens pos0 .. pos0 + R - 1 of a cache
                    // of T tokens); 0 for a whole-sequence prefill
    int qps;        // decode: queries per sequence (multi-token decode).  B then counts queries: query b belongs to
                    // cache sequence b / qps and is its token number b % qps of the qps newest ones; 1 otherwise
};

__host__ __device__ inline int floordiv_i(int a, int b) {
    int q = a / b;
    if ((a % b != 0) && ((a < 0) != (b < 0))) --q;
    return q;
}

// Left edge of the chunk-aligned local window (Sec. 2.1), clamped at 0.
__host__ __device__ inline int local_lo(int pos, int W, int S) {
    int lo = floordiv_i(pos - W + 1, S) * S;
    return lo < 0 ? 0 : lo;
}

__device__ inline float to_f32(float x) { return x; }
__device__ inline float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ inline T from_f32(float x);
template <> __device__ inline float from_f32<float>(float x) { return x; }
template <> __device__ inline __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// 8 consecutive elements (16-byte aligned for bf16, 32-byte for fp32) widened to fp32.
__device__ inline void load8(const float* p, float (&x)[8]) {
    const float4 a = *reinterpret_cast<const float4*>(p);
    const float4 b = *reinterpret_cast<const float4*>(p + 4);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
    x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
__device__ inline void load8(const __nv_bfloat16* p, float (&x)[8]) {
    const uint4 raw = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        x[2 * i] = __uint_as_float(w[i] << 16);
        x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

// Order-preserving map fp32 -> uint32 (larger float -> larger key); -0 is folded into +0 first.
__device__ inline uint32_t ordered_key(float s) {
    s += 0.0f;
    const uint32_t u = __float_as_uint(s);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ inline float key_to_float(uint32_t k) {
    const uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
    return __uint_as_float(u);
}
// 64-bit selection key: score first, then the LOWER chunk id wins.  Never 0 for a valid chunk.
__device__ inline unsigned long long select_key(float score, int chunk) {
    return (static_cast<unsigned long long>(ordered_key(score)) << 32) |
           static_cast<unsigned long long>(0xffffffffu - static_cast<uint32_t>(chunk));
}
__device__ inline int key_chunk(unsigned long long key) {
    return static_cast<int>(0xffffffffu - static_cast<uint32_t>(key & 0xffffffffull));
}

__device__ inline float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFullMask, v, o));
    return v;
}
__device__ inline float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFullMask, v, o);
    return v;
}

// Access policy of the prefill partial-output buffer (written once by the attend kernel, read once by the
// fuse kernel).  Default: streaming (evict-first) both ways, so that the buffer does not push the gathered
// queries out of L2.  -DHILS_OBUF_CACHED keeps it under the normal policy (for query blocks small enough that the
// whole buffer stays L2-resident between the two kernels).
__device__ inline void obuf_store(uint4* p, const uint4& v) {
#ifdef HILS_OBUF_CACHED
    *p = v;
#else
    __stcs(p, v);
#endif
}
__device__ inline uint4 obuf_load(const uint4* p) {
#ifdef HILS_OBUF_CACHED
    return *p;
#else
    return __ldcs(p);
#endif
}

__device__ inline void set_status(int* status, int code) {
    if (status) atomicCAS(status, 0, code);
}

}  // namespace hils
