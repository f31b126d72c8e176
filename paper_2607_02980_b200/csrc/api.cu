// C ABI of the HiLS library: argument validation, kernel-set dispatch, host-buffer variants.
#include <string.h>

#include <mutex>
#include <vector>

#include "internal.h"

namespace hils {
namespace {

thread_local int g_last_launches = 0;

constexpr int kMaxTrace = 1024;
struct Trace {
    bool enabled = false;
    bool have_events = false;
    cudaEvent_t ev[kMaxTrace + 1];
    const char* names[kMaxTrace];
    int n = 0;
};
thread_local Trace g_trace;

}  // namespace

int sm_count() {
    // per device, looked up once; 148 (B200) where no device answers, e.g. a workspace-size query on a host without a GPU
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

void trace_begin(cudaStream_t stream) {
    Trace& t = g_trace;
    t.n = 0;
    if (t.enabled && t.have_events) cudaEventRecord(t.ev[0], stream);
}

bool trace_active() { return g_trace.enabled && g_trace.have_events; }

void trace_mark(const char* name, cudaStream_t stream) {
    Trace& t = g_trace;
    if (!t.enabled || !t.have_events || t.n >= kMaxTrace) return;
    t.names[t.n] = name;
    ++t.n;
    cudaEventRecord(t.ev[t.n], stream);
}

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline size_t elem_bytes(int dtype) { return dtype == HILS_F32 ? 4 : 2; }

// Fills `s` from the public parameters; returns a status.
int make_shape(const hils_params* p, int is_decode, Shape* s, long long pos0 = 0) {
    if (!p) return HILS_ERR_INVALID_ARG;
    if (p->B < 1 || p->Hq < 1 || p->Hkv < 1 || p->d < 1 || p->chunk_size < 1 || p->top_k < 1 || p->window < 1)
        return HILS_ERR_INVALID_ARG;
    if (p->Hq % p->Hkv != 0) return HILS_ERR_INVALID_ARG;
    if (p->Hl != p->Hkv && p->Hl != p->Hq) return HILS_ERR_INVALID_ARG;
    if (p->dtype != HILS_F32 && p->dtype != HILS_BF16) return HILS_ERR_INVALID_ARG;
    if (p->impl < HILS_IMPL_AUTO || p->impl > HILS_IMPL_PACKED) return HILS_ERR_INVALID_ARG;
    if (!(p->scale >= 0.f)) return HILS_ERR_INVALID_ARG;
    s->B = p->B; s->Hq = p->Hq; s->Hkv = p->Hkv; s->Hl = p->Hl; s->G = p->Hq / p->Hkv;
    s->d = p->d; s->S = p->chunk_size; s->K = p->top_k; s->W = p->window;
    s->scale = p->scale > 0.f ? p->scale : 1.0f / sqrtf(static_cast<float>(p->d));
    s->is_decode = is_decode;
    s->pos0 = 0;
    s->qps = 1;
    if (is_decode) {
        if (p->T_max < 1) return HILS_ERR_INVALID_ARG;
        s->R = 1;
        s->T = p->T_max;
    } else {
        if (p->L < 1) return HILS_ERR_INVALID_ARG;
        s->R = p->L;
        s->T = p->T_max > 0 ? p->T_max : p->L;
        if (pos0 < 0 || pos0 + p->L > s->T) return HILS_ERR_INVALID_ARG;      // the cache holds the queries' tokens
        s->pos0 = static_cast<int>(pos0);
    }
    s->C = p->C > 0 ? p->C : s->T / s->S;
    // every candidate chunk of the last position must have a landmark row
    const int last = is_decode ? s->T - 1 : s->pos0 + p->L - 1;
    const int max_cand = local_lo(last, s->W, s->S) / s->S;
    if (s->C < max_cand) return HILS_ERR_INVALID_ARG;
    return HILS_OK;
}

enum class Path { Generic, DecodeFast, PrefillFast, PrefillPacked };

int pick_path(const Shape& s, const hils_params* p, Path* path) {
    const bool fast_ok = s.is_decode ? decode_fast_supports(s, p->dtype) : prefill_fast_supports(s, p->dtype);
    if (p->impl == HILS_IMPL_PACKED) {
        if (s.is_decode || !prefill_packed_supports(s, p->dtype)) return HILS_ERR_UNSUPPORTED;
        *path = Path::PrefillPacked;
        return HILS_OK;
    }
    if (p->impl == HILS_IMPL_FAST) {
        if (!fast_ok) return HILS_ERR_UNSUPPORTED;
        *path = s.is_decode ? Path::DecodeFast : Path::PrefillFast;
        return HILS_OK;
    }
    if (p->impl == HILS_IMPL_AUTO && fast_ok) {
        *path = s.is_decode ? Path::DecodeFast : Path::PrefillFast;
        return HILS_OK;
    }
    if (!generic_supports(s)) return HILS_ERR_UNSUPPORTED;
    *path = Path::Generic;
    return HILS_OK;
}

size_t scratch_bytes(const Shape& s, Path path) {
    switch (path) {
        case Path::DecodeFast: return decode_fast_scratch_bytes(s);
        case Path::PrefillFast: return prefill_fast_scratch_bytes(s);
        default: return 0;
    }
}

int run(const hils_params* p, int is_decode, const void* q, const void* k, const void* v, const void* lm,
        const float* bias, const int32_t* seq_lens, void* out, float* lse, int32_t* sel, void* ws,
        size_t ws_bytes, void* stream_v, const int32_t* block_table = nullptr, int num_pages = 0, long long pos0 = 0,
        const void* q_route = nullptr, int qps = 1) {
    g_last_launches = 0;
    Shape s;
    int rc = make_shape(p, is_decode, &s, pos0);
    if (rc != HILS_OK) return rc;
    if (qps != 1) {
        // multi-token decode: qps queries per sequence, run as B * qps decode queries over shared caches
        if (!is_decode || qps < 1 || static_cast<long long>(s.B) * qps > (1 << 24)) return HILS_ERR_INVALID_ARG;
        s.B *= qps;
        s.qps = qps;
    }
    if (!q || !k || !v || !lm || !out || !lse || !sel || (is_decode && !seq_lens)) return HILS_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(lm) || !aligned16(out) ||
        (reinterpret_cast<uintptr_t>(lse) & 3u) || (reinterpret_cast<uintptr_t>(sel) & 3u) ||
        (bias && (reinterpret_cast<uintptr_t>(bias) & 3u)))
        return HILS_ERR_ALIGNMENT;
    Path path;
    rc = pick_path(s, p, &path);
    if (rc != HILS_OK) return rc;
    if (qps != 1 && path != Path::DecodeFast) return HILS_ERR_UNSUPPORTED;     // shared caches: TMA decode kernels only
    if (block_table) {
        // paged caches: only the TMA decode kernels address K / V through a page table
        if (path != Path::DecodeFast) return HILS_ERR_UNSUPPORTED;
        if (num_pages < 1 || static_cast<long long>(num_pages) * s.Hkv * s.S >= (1ll << 31)) return HILS_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(block_table) & 3u) return HILS_ERR_ALIGNMENT;
    }
    const size_t need = kStatusBytes + scratch_bytes(s, path);
    if (!ws || ws_bytes < need) return HILS_ERR_WORKSPACE;
    if (!aligned16(ws)) return HILS_ERR_ALIGNMENT;
    Tensors t{q, k, v, lm, bias, seq_lens, out, lse, sel, static_cast<int*>(ws),
              static_cast<char*>(ws) + kStatusBytes, ws_bytes - kStatusBytes};
    t.block_table = block_table;
    t.num_pages = num_pages;
    if (q_route && !aligned16(q_route)) return HILS_ERR_ALIGNMENT;
    t.q_route = q_route;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    trace_begin(stream);
    int n;
    switch (path) {
        case Path::DecodeFast: n = launch_decode_fast(s, t, stream); break;
        case Path::PrefillFast: n = launch_prefill_fast(s, t, stream); break;
        case Path::PrefillPacked: n = launch_prefill_packed(s, t, stream); break;
        default: n = launch_generic(s, p->dtype, t, stream); break;
    }
    if (n < 0) return n;
    g_last_launches = n;
    return HILS_OK;
}

struct ArenaLayout {
    size_t q, k, v, lm, bias, seq, out, lse, sel, ws, total;
    size_t q_b, kv_b, lm_b, bias_b, seq_b, out_b, lse_b, sel_b, ws_b;
};

int arena_layout(const hils_params* p, int is_decode, ArenaLayout* a) {
    Shape s;
    int rc = make_shape(p, is_decode, &s);
    if (rc != HILS_OK) return rc;
    const size_t eb = elem_bytes(p->dtype);
    const size_t rows = static_cast<size_t>(s.B) * s.Hq * s.R;
    a->q_b = rows * s.d * eb;
    a->kv_b = static_cast<size_t>(s.B) * s.Hkv * s.T * s.d * eb;
    a->lm_b = static_cast<size_t>(s.B) * s.Hl * s.C * s.d * eb;
    a->bias_b = static_cast<size_t>(s.B) * s.Hl * s.C * 4;
    a->seq_b = static_cast<size_t>(s.B) * 4;
    a->out_b = a->q_b;
    a->lse_b = rows * 4;
    a->sel_b = static_cast<size_t>(s.B) * s.Hkv * s.R * s.K * 4;
    a->ws_b = hils_workspace_bytes(p, is_decode);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    a->ws = take(a->ws_b);        // first, so that the arena's head is the status word
    a->q = take(a->q_b); a->k = take(a->kv_b); a->v = take(a->kv_b); a->lm = take(a->lm_b);
    a->bias = take(a->bias_b); a->seq = take(a->seq_b); a->out = take(a->out_b);
    a->lse = take(a->lse_b); a->sel = take(a->sel_b);
    a->total = off;
    return HILS_OK;
}

// ---- pipelined host-buffer prefill -------------------------------------------------------------------------
// The operator is causal, so a block of query tokens needs only the inputs up to its own end: blocks of
// kHostBlock tokens are copied in, computed (the slice entry point) and copied out on three internal streams,
// and the transfers of neighbouring blocks overlap each other (PCIe is full duplex) and the kernels.
#ifndef HILS_HOST_BLOCK
#define HILS_HOST_BLOCK 4096
#endif
constexpr int kHostBlock = HILS_HOST_BLOCK;

struct HostPipe {
    bool ok = false;
    cudaStream_t in = nullptr, cmp = nullptr, out = nullptr;
    cudaEvent_t fork = nullptr, in_done[2] = {nullptr, nullptr}, cmp_done[2] = {nullptr, nullptr},
                out_done[2] = {nullptr, nullptr}, tail[3] = {nullptr, nullptr, nullptr};
};
std::mutex g_pipe_mutex;       // the events are shared: calls that enqueue through the pipe are serialised on the host
HostPipe g_pipe[64];

HostPipe* host_pipe() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    HostPipe& hp = g_pipe[dev];
    if (!hp.ok) {
        auto mk = [](cudaEvent_t* e) { return cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess; };
        if (cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&hp.cmp, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) != cudaSuccess)
            return nullptr;
        bool good = mk(&hp.fork);
        for (int i = 0; i < 2; ++i) good = good && mk(&hp.in_done[i]) && mk(&hp.cmp_done[i]) && mk(&hp.out_done[i]);
        for (int i = 0; i < 3; ++i) good = good && mk(&hp.tail[i]);
        if (!good) return nullptr;
        hp.ok = true;
    }
    return &hp;
}

// Returns HILS_OK, an error, or 1 when the pipelined form does not apply (the caller then takes the plain path).
int run_host_prefill_pipelined(const hils_params* p, const ArenaLayout& full, const void* q, const void* k,
                               const void* v, const void* lm, const float* bias, void* out, float* lse, int32_t* sel,
                               char* base, void* stream_v) {
    static const bool off = [] { const char* e = getenv("HILS_HOST_PIPELINE"); return e && e[0] == '0'; }();
    if (off || p->L < 2 * kHostBlock || (p->T_max > 0 && p->T_max != p->L) || trace_active()) return 1;
    Shape s;
    if (make_shape(p, 0, &s) != HILS_OK) return 1;
    const size_t eb = elem_bytes(p->dtype);
    const int L = p->L;
    // Block schedule: kHostBlock tokens each, the last stretch in shrinking pieces (1/2, 1/4, 1/4): what cannot
    // overlap anything is the last block's compute and copy-out, so that block is kept short.
    std::vector<int> blk_i0, blk_len;
    {
        int i0 = 0;
        while (L - i0 > kHostBlock) { blk_i0.push_back(i0); blk_len.push_back(kHostBlock); i0 += kHostBlock; }
        const int rem = L - i0;
        const int half = (rem / 2 + 63) / 64 * 64, quarter = (rem / 4 + 63) / 64 * 64;
        int cuts[3] = {half, quarter, rem};
        for (int c = 0; c < 3 && i0 < L; ++c) {
            const int len = c == 2 ? L - i0 : (cuts[c] < L - i0 ? cuts[c] : L - i0);
            if (len <= 0) continue;
            blk_i0.push_back(i0);
            blk_len.push_back(len);
            i0 += len;
        }
    }
    const int nb = static_cast<int>(blk_i0.size());
    hils_params bp = *p;
    bp.T_max = L;
    size_t ws_b = 0;
    for (int b = 0; b < nb; ++b) {
        bp.L = blk_len[b];
        const size_t need = hils_prefill_at_workspace_bytes(&bp, blk_i0[b]);
        if (need == 0) return 1;
        ws_b = need > ws_b ? need : ws_b;
    }
    // layout inside the caller's arena: workspace, K, V, landmarks, bias, then two slots of per-block q / out / lse / sel
    const size_t rowsq = static_cast<size_t>(s.B) * s.Hq, rowskv = static_cast<size_t>(s.B) * s.Hkv;
    const size_t q_blk = rowsq * kHostBlock * s.d * eb, lse_blk = rowsq * kHostBlock * 4;
    const size_t sel_blk = rowskv * kHostBlock * s.K * 4;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    const size_t a_ws = take(ws_b), a_k = take(full.kv_b), a_v = take(full.kv_b), a_lm = take(full.lm_b), a_bias = take(full.bias_b);
    size_t a_q[2], a_out[2], a_lse[2], a_sel[2];
    for (int i = 0; i < 2; ++i) { a_q[i] = take(q_blk); a_out[i] = take(q_blk); a_lse[i] = take(lse_blk); a_sel[i] = take(sel_blk); }
    if (o > full.total) return 1;

    std::lock_guard<std::mutex> lock(g_pipe_mutex);
    HostPipe* hp = host_pipe();
    if (!hp) return 1;
    cudaStream_t user = static_cast<cudaStream_t>(stream_v);
    bool ok = cudaEventRecord(hp->fork, user) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(hp->in, hp->fork, 0) == cudaSuccess && cudaStreamWaitEvent(hp->cmp, hp->fork, 0) == cudaSuccess &&
         cudaStreamWaitEvent(hp->out, hp->fork, 0) == cudaSuccess;
    // the status word at the arena's head stays as the caller left it; landmarks and bias go first
    ok = ok && cudaMemcpyAsync(base + a_lm, lm, full.lm_b, cudaMemcpyHostToDevice, hp->in) == cudaSuccess;
    if (bias) ok = ok && cudaMemcpyAsync(base + a_bias, bias, full.bias_b, cudaMemcpyHostToDevice, hp->in) == cudaSuccess;
    if (!ok) return HILS_ERR_CUDA;
    int launches = 0;
    const size_t tok_b = static_cast<size_t>(s.d) * eb;                  // bytes per token row
    for (int b = 0; b < nb; ++b) {
        const int i0 = blk_i0[b], len = blk_len[b], sl = b & 1;
        // ---- copy in: this block's K / V rows into the device caches, its queries into slot sl
        if (b >= 2) ok = ok && cudaStreamWaitEvent(hp->in, hp->cmp_done[sl], 0) == cudaSuccess;
        ok = ok && cudaMemcpy2DAsync(base + a_k + i0 * tok_b, L * tok_b, static_cast<const char*>(k) + i0 * tok_b, L * tok_b,
                                     len * tok_b, rowskv, cudaMemcpyHostToDevice, hp->in) == cudaSuccess;
        ok = ok && cudaMemcpy2DAsync(base + a_v + i0 * tok_b, L * tok_b, static_cast<const char*>(v) + i0 * tok_b, L * tok_b,
                                     len * tok_b, rowskv, cudaMemcpyHostToDevice, hp->in) == cudaSuccess;
        ok = ok && cudaMemcpy2DAsync(base + a_q[sl], len * tok_b, static_cast<const char*>(q) + i0 * tok_b, L * tok_b,
                                     len * tok_b, rowsq, cudaMemcpyHostToDevice, hp->in) == cudaSuccess;
        ok = ok && cudaEventRecord(hp->in_done[sl], hp->in) == cudaSuccess;
        // ---- compute
        ok = ok && cudaStreamWaitEvent(hp->cmp, hp->in_done[sl], 0) == cudaSuccess;
        if (b >= 2) ok = ok && cudaStreamWaitEvent(hp->cmp, hp->out_done[sl], 0) == cudaSuccess;
        if (!ok) return HILS_ERR_CUDA;
        bp.L = len;
        const int rc = run(&bp, 0, base + a_q[sl], base + a_k, base + a_v, base + a_lm,
                           bias ? reinterpret_cast<const float*>(base + a_bias) : nullptr, nullptr, base + a_out[sl],
                           reinterpret_cast<float*>(base + a_lse[sl]), reinterpret_cast<int32_t*>(base + a_sel[sl]),
                           base + a_ws, ws_b, hp->cmp, nullptr, 0, i0);
        if (rc != HILS_OK) return rc;
        launches += g_last_launches;
        ok = ok && cudaEventRecord(hp->cmp_done[sl], hp->cmp) == cudaSuccess;
        // ---- copy out
        ok = ok && cudaStreamWaitEvent(hp->out, hp->cmp_done[sl], 0) == cudaSuccess;
        ok = ok && cudaMemcpy2DAsync(static_cast<char*>(out) + i0 * tok_b, L * tok_b, base + a_out[sl], len * tok_b, len * tok_b,
                                     rowsq, cudaMemcpyDeviceToHost, hp->out) == cudaSuccess;
        ok = ok && cudaMemcpy2DAsync(reinterpret_cast<char*>(lse) + static_cast<size_t>(i0) * 4, static_cast<size_t>(L) * 4,
                                     base + a_lse[sl], static_cast<size_t>(len) * 4, static_cast<size_t>(len) * 4, rowsq,
                                     cudaMemcpyDeviceToHost, hp->out) == cudaSuccess;
        const size_t selrow = static_cast<size_t>(s.K) * 4;
        ok = ok && cudaMemcpy2DAsync(reinterpret_cast<char*>(sel) + i0 * selrow, L * selrow, base + a_sel[sl], len * selrow,
                                     len * selrow, rowskv, cudaMemcpyDeviceToHost, hp->out) == cudaSuccess;
        ok = ok && cudaEventRecord(hp->out_done[sl], hp->out) == cudaSuccess;
        if (!ok) return HILS_ERR_CUDA;
    }
    // ---- join: the caller's stream continues after everything enqueued here
    ok = ok && cudaEventRecord(hp->tail[0], hp->in) == cudaSuccess && cudaEventRecord(hp->tail[1], hp->cmp) == cudaSuccess &&
         cudaEventRecord(hp->tail[2], hp->out) == cudaSuccess;
    for (int i = 0; i < 3; ++i) ok = ok && cudaStreamWaitEvent(user, hp->tail[i], 0) == cudaSuccess;
    g_last_launches = launches;
    return ok ? HILS_OK : HILS_ERR_CUDA;
}

int run_host(const hils_params* p, int is_decode, const void* q, const void* k, const void* v, const void* lm,
             const float* bias, const int32_t* seq_lens, void* out, float* lse, int32_t* sel, void* arena,
             size_t arena_bytes, void* stream_v) {
    ArenaLayout a;
    int rc = arena_layout(p, is_decode, &a);
    if (rc != HILS_OK) return rc;
    if (!q || !k || !v || !lm || !out || !lse || !sel || (is_decode && !seq_lens)) return HILS_ERR_INVALID_ARG;
    if (!arena || arena_bytes < a.total) return HILS_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(arena) & 255u) return HILS_ERR_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    char* base = static_cast<char*>(arena);
    if (!is_decode) {
        rc = run_host_prefill_pipelined(p, a, q, k, v, lm, bias, out, lse, sel, base, stream_v);
        if (rc != 1) return rc;
    }
    bool ok = true;
    ok &= cudaMemcpyAsync(base + a.q, q, a.q_b, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(base + a.k, k, a.kv_b, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(base + a.v, v, a.kv_b, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(base + a.lm, lm, a.lm_b, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    if (bias) ok &= cudaMemcpyAsync(base + a.bias, bias, a.bias_b, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    if (is_decode)
        ok &= cudaMemcpyAsync(base + a.seq, seq_lens, a.seq_b, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    if (!ok) return HILS_ERR_CUDA;
    rc = run(p, is_decode, base + a.q, base + a.k, base + a.v, base + a.lm,
             bias ? reinterpret_cast<const float*>(base + a.bias) : nullptr,
             is_decode ? reinterpret_cast<const int32_t*>(base + a.seq) : nullptr, base + a.out,
             reinterpret_cast<float*>(base + a.lse), reinterpret_cast<int32_t*>(base + a.sel), base + a.ws,
             a.ws_b, stream_v);
    if (rc != HILS_OK) return rc;
    ok &= cudaMemcpyAsync(out, base + a.out, a.out_b, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(lse, base + a.lse, a.lse_b, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(sel, base + a.sel, a.sel_b, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    return ok ? HILS_OK : HILS_ERR_CUDA;
}

}  // namespace
}  // namespace hils

using namespace hils;

extern "C" {

size_t hils_workspace_bytes(const hils_params* params, int is_decode) {
    Shape s;
    if (make_shape(params, is_decode, &s) != HILS_OK) return 0;
    Path path;
    if (pick_path(s, params, &path) != HILS_OK) return 0;
    return kStatusBytes + align_up(scratch_bytes(s, path), 256);
}

int hils_prefill(const hils_params* params, const void* q, const void* k, const void* v, const void* landmarks,
                 const float* bias, void* out, float* lse, int32_t* sel_idx, void* workspace,
                 size_t workspace_bytes, void* stream) {
    return run(params, 0, q, k, v, landmarks, bias, nullptr, out, lse, sel_idx, workspace, workspace_bytes, stream);
}

int hils_decode(const hils_params* params, const void* q, const void* k_cache, const void* v_cache,
                const void* landmarks, const float* bias, const int32_t* seq_lens, void* out, float* lse,
                int32_t* sel_idx, void* workspace, size_t workspace_bytes, void* stream) {
    return run(params, 1, q, k_cache, v_cache, landmarks, bias, seq_lens, out, lse, sel_idx, workspace,
               workspace_bytes, stream);
}

int hils_prefill_routed(const hils_params* params, const void* q, const void* q_route, const void* k, const void* v,
                        const void* landmarks, const float* bias, void* out, float* lse, int32_t* sel_idx,
                        void* workspace, size_t workspace_bytes, void* stream) {
    if (!q_route) return HILS_ERR_INVALID_ARG;
    return run(params, 0, q, k, v, landmarks, bias, nullptr, out, lse, sel_idx, workspace, workspace_bytes, stream,
               nullptr, 0, 0, q_route);
}

int hils_decode_routed(const hils_params* params, const void* q, const void* q_route, const void* k_cache,
                       const void* v_cache, const void* landmarks, const float* bias, const int32_t* seq_lens,
                       void* out, float* lse, int32_t* sel_idx, void* workspace, size_t workspace_bytes,
                       void* stream) {
    if (!q_route) return HILS_ERR_INVALID_ARG;
    return run(params, 1, q, k_cache, v_cache, landmarks, bias, seq_lens, out, lse, sel_idx, workspace,
               workspace_bytes, stream, nullptr, 0, 0, q_route);
}

int hils_prefill_at(const hils_params* params, const void* q, const void* k, const void* v, const void* landmarks,
                    const float* bias, int64_t pos0, void* out, float* lse, int32_t* sel_idx, void* workspace,
                    size_t workspace_bytes, void* stream) {
    return run(params, 0, q, k, v, landmarks, bias, nullptr, out, lse, sel_idx, workspace, workspace_bytes, stream,
               nullptr, 0, pos0);
}

size_t hils_prefill_at_workspace_bytes(const hils_params* params, int64_t pos0) {
    Shape s;
    if (make_shape(params, 0, &s, pos0) != HILS_OK) return 0;
    Path path;
    if (pick_path(s, params, &path) != HILS_OK) return 0;
    return kStatusBytes + align_up(scratch_bytes(s, path), 256);
}

int hils_decode_paged(const hils_params* params, const void* q, const void* k_pages, const void* v_pages,
                      const void* landmarks, const float* bias, const int32_t* block_table, int32_t num_pages,
                      const int32_t* seq_lens, void* out, float* lse, int32_t* sel_idx, void* workspace,
                      size_t workspace_bytes, void* stream) {
    if (!block_table) return HILS_ERR_INVALID_ARG;
    return run(params, 1, q, k_pages, v_pages, landmarks, bias, seq_lens, out, lse, sel_idx, workspace, workspace_bytes,
               stream, block_table, num_pages);
}

size_t hils_decode_multi_workspace_bytes(const hils_params* params, int32_t tokens_per_seq) {
    Shape s;
    if (tokens_per_seq < 1 || make_shape(params, 1, &s) != HILS_OK) return 0;
    if (static_cast<long long>(s.B) * tokens_per_seq > (1 << 24)) return 0;
    s.B *= tokens_per_seq;
    s.qps = tokens_per_seq;
    if (params->impl == HILS_IMPL_GENERIC || !decode_fast_supports(s, params->dtype)) return 0;
    return kStatusBytes + align_up(decode_fast_scratch_bytes(s), 256);
}

int hils_decode_multi(const hils_params* params, int32_t tokens_per_seq, const void* q, const void* k_cache,
                      const void* v_cache, const void* landmarks, const float* bias, const int32_t* block_table,
                      int32_t num_pages, const int32_t* seq_lens, void* out, float* lse, int32_t* sel_idx,
                      void* workspace, size_t workspace_bytes, void* stream) {
    if (tokens_per_seq < 1) return HILS_ERR_INVALID_ARG;
    if (params && params->impl == HILS_IMPL_GENERIC) return HILS_ERR_UNSUPPORTED;
    return run(params, 1, q, k_cache, v_cache, landmarks, bias, seq_lens, out, lse, sel_idx, workspace, workspace_bytes,
               stream, block_table, num_pages, 0, nullptr, tokens_per_seq);
}

int hils_decode_noalloc(const hils_params* params, const void* q, const void* k_cache, const void* v_cache,
                        const void* landmarks, const float* bias, const int32_t* seq_lens, void* out, float* lse,
                        int32_t* sel_idx, int32_t* device_status, void* stream) {
    g_last_launches = 0;
    Shape s;
    int rc = make_shape(params, 1, &s);
    if (rc != HILS_OK) return rc;
    if (!q || !k_cache || !v_cache || !landmarks || !seq_lens || !out || !lse || !sel_idx) return HILS_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(landmarks) || !aligned16(out) ||
        (reinterpret_cast<uintptr_t>(lse) & 3u) || (reinterpret_cast<uintptr_t>(sel_idx) & 3u) ||
        (bias && (reinterpret_cast<uintptr_t>(bias) & 3u)) ||
        (device_status && (reinterpret_cast<uintptr_t>(device_status) & 3u)))
        return HILS_ERR_ALIGNMENT;
    if (!decode_fast_supports(s, params->dtype)) return HILS_ERR_UNSUPPORTED;
    Tensors t{q, k_cache, v_cache, landmarks, bias, seq_lens, out, lse, sel_idx, nullptr, nullptr, 0};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    trace_begin(st);
    const int n = launch_decode_noalloc(s, t, device_status, st);
    if (n < 0) return n;
    g_last_launches = n;
    return HILS_OK;
}

int hils_landmark_summary(const hils_params* params, const void* landmark_queries, const void* k,
                          const int32_t* seq_lens, int32_t chunk_begin, int32_t chunk_count, void* landmarks,
                          float* bias, void* stream) {
    g_last_launches = 0;
    const hils_params* p = params;
    if (!p || !landmark_queries || !k || !landmarks || !bias) return HILS_ERR_INVALID_ARG;
    if (p->B < 1 || p->Hkv < 1 || p->Hl < 1 || p->Hl % p->Hkv != 0 || p->C < 1 || p->d < 1 || p->chunk_size < 1)
        return HILS_ERR_INVALID_ARG;
    if (p->dtype != HILS_F32 && p->dtype != HILS_BF16) return HILS_ERR_INVALID_ARG;
    const long long T = p->T_max > 0 ? p->T_max : p->L;
    if (T < 1 || !(p->scale >= 0.f)) return HILS_ERR_INVALID_ARG;
    if (chunk_begin < 0 || chunk_begin > p->C) return HILS_ERR_INVALID_ARG;
    const int cn = chunk_count <= 0 ? p->C - chunk_begin : chunk_count;
    if (cn > p->C - chunk_begin) return HILS_ERR_INVALID_ARG;
    if (!aligned16(landmark_queries) || !aligned16(k) || !aligned16(landmarks) ||
        (reinterpret_cast<uintptr_t>(bias) & 3u) || (seq_lens && (reinterpret_cast<uintptr_t>(seq_lens) & 3u)))
        return HILS_ERR_ALIGNMENT;
    if (!landmark_summary_supports(p->d, p->chunk_size)) return HILS_ERR_UNSUPPORTED;
    const float scale = p->scale > 0.f ? p->scale : 1.0f / sqrtf(static_cast<float>(p->d));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    trace_begin(st);
    const int n = launch_landmark_summary(p->dtype, p->B, p->Hkv, p->Hl, p->C, p->d, p->chunk_size, T, scale,
                                          landmark_queries, k, seq_lens, chunk_begin, cn, landmarks, bias, st);
    if (n < 0) return n;
    trace_mark("landmark_summary", st);
    g_last_launches = n;
    return HILS_OK;
}

size_t hils_prefill_backward_workspace_bytes(const hils_params* params) {
    Shape s;
    if (make_shape(params, 0, &s) != HILS_OK) return 0;
    const bool fast = params->impl != HILS_IMPL_GENERIC && prefill_backward_fast_supports(s, params->dtype);
    if (fast) return kStatusBytes + prefill_backward_fast_scratch_bytes(s);
    if (params->impl == HILS_IMPL_FAST || !generic_supports(s)) return 0;
    return kStatusBytes;
}

int hils_prefill_backward(const hils_params* params, const void* q, const void* k, const void* v,
                          const void* landmarks, const float* bias, const void* out, const float* lse,
                          const int32_t* sel_idx, const void* dout, float* dq, float* dk, float* dv,
                          float* dlandmarks, float* dbias, void* workspace, size_t workspace_bytes, void* stream) {
    g_last_launches = 0;
    const hils_params* p = params;
    Shape s;
    int rc = make_shape(p, 0, &s);
    if (rc != HILS_OK) return rc;
    if (!q || !k || !v || !landmarks || !out || !lse || !sel_idx || !dout || !dq || !dk || !dv || !dlandmarks)
        return HILS_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(landmarks) || !aligned16(out) ||
        !aligned16(dout) || !aligned16(dq) || !aligned16(dk) || !aligned16(dv) || !aligned16(dlandmarks) ||
        (reinterpret_cast<uintptr_t>(lse) & 3u) || (reinterpret_cast<uintptr_t>(sel_idx) & 3u) ||
        (bias && (reinterpret_cast<uintptr_t>(bias) & 3u)) || (dbias && (reinterpret_cast<uintptr_t>(dbias) & 3u)))
        return HILS_ERR_ALIGNMENT;
    const bool fast = p->impl != HILS_IMPL_GENERIC && prefill_backward_fast_supports(s, p->dtype);
    if (!fast && (p->impl == HILS_IMPL_FAST || !generic_supports(s))) return HILS_ERR_UNSUPPORTED;
    const size_t need = hils_prefill_backward_workspace_bytes(p);
    if (!workspace || workspace_bytes < need) return HILS_ERR_WORKSPACE;
    if (!aligned16(workspace)) return HILS_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the four shared gradients are accumulated: they start at zero (dq is written whole)
    const size_t kv = static_cast<size_t>(s.B) * s.Hkv * s.T * s.d * sizeof(float);
    const size_t lmb = static_cast<size_t>(s.B) * s.Hl * s.C * sizeof(float);
    if (cudaMemsetAsync(dk, 0, kv, st) != cudaSuccess || cudaMemsetAsync(dv, 0, kv, st) != cudaSuccess ||
        cudaMemsetAsync(dlandmarks, 0, lmb * s.d, st) != cudaSuccess ||
        (dbias && cudaMemsetAsync(dbias, 0, lmb, st) != cudaSuccess))
        return HILS_ERR_CUDA;
    BackwardTensors t{q, k, v, landmarks, bias, out, lse, sel_idx, dout, dq, dk, dv, dlandmarks, dbias,
                      static_cast<int*>(workspace), static_cast<char*>(workspace) + kStatusBytes,
                      workspace_bytes - kStatusBytes};
    trace_begin(st);
    int n;
    if (fast) {
        // dq is accumulated too on this path (one reduction per slot of a row)
        if (cudaMemsetAsync(dq, 0, static_cast<size_t>(s.B) * s.Hq * s.R * s.d * sizeof(float), st) != cudaSuccess)
            return HILS_ERR_CUDA;
        n = launch_prefill_backward_fast(s, t, st);
    } else {
        n = launch_backward_generic(s, p->dtype, t, st);
    }
    if (n < 0) return n;
    g_last_launches = n;
    return HILS_OK;
}

int hils_chunk_overlap(const hils_params* params, const int32_t* sel_idx, int32_t block_queries, int32_t* stats,
                       float* overlap, void* stream) {
    g_last_launches = 0;
    const hils_params* p = params;
    if (!p || !sel_idx || !stats) return HILS_ERR_INVALID_ARG;
    if (p->B < 1 || p->Hkv < 1 || p->L < 1 || p->C < 1 || p->top_k < 1 || block_queries < 1)
        return HILS_ERR_INVALID_ARG;
    if (static_cast<long long>(block_queries) * p->top_k > (1ll << 24)) return HILS_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(sel_idx) & 3u) || (reinterpret_cast<uintptr_t>(stats) & 15u) ||
        (overlap && (reinterpret_cast<uintptr_t>(overlap) & 3u)))
        return HILS_ERR_ALIGNMENT;
    if (!chunk_overlap_supports(p->C)) return HILS_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    trace_begin(st);
    const int n = launch_chunk_overlap(p->B * p->Hkv, p->L, p->top_k, p->C, block_queries, sel_idx, stats, overlap, st);
    if (n < 0) return n;
    trace_mark("chunk_overlap", st);
    g_last_launches = n;
    return HILS_OK;
}

size_t hils_host_arena_bytes(const hils_params* params, int is_decode) {
    ArenaLayout a;
    if (arena_layout(params, is_decode, &a) != HILS_OK || a.ws_b == 0) return 0;
    return a.total;
}

int hils_prefill_host(const hils_params* params, const void* q_host, const void* k_host, const void* v_host,
                      const void* landmarks_host, const float* bias_host, void* out_host, float* lse_host,
                      int32_t* sel_idx_host, void* device_arena, size_t arena_bytes, void* stream) {
    return run_host(params, 0, q_host, k_host, v_host, landmarks_host, bias_host, nullptr, out_host, lse_host,
                    sel_idx_host, device_arena, arena_bytes, stream);
}

int hils_decode_host(const hils_params* params, const void* q_host, const void* k_cache_host,
                     const void* v_cache_host, const void* landmarks_host, const float* bias_host,
                     const int32_t* seq_lens_host, void* out_host, float* lse_host, int32_t* sel_idx_host,
                     void* device_arena, size_t arena_bytes, void* stream) {
    return run_host(params, 1, q_host, k_cache_host, v_cache_host, landmarks_host, bias_host, seq_lens_host,
                    out_host, lse_host, sel_idx_host, device_arena, arena_bytes, stream);
}

int hils_poll_status(const void* workspace, void* stream) {
    if (!workspace) return HILS_ERR_INVALID_ARG;
    int word = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return HILS_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return HILS_ERR_CUDA;
    if (word == 0) return HILS_OK;
    if (word == kDevTimeout) return HILS_ERR_DEVICE_TIMEOUT;
    if (word == kDevBadIndex) return HILS_ERR_DEVICE_INDEX;
    return HILS_ERR_CUDA;
}

int hils_last_launch_count(void) { return g_last_launches; }

int hils_trace_enable(int on) {
    Trace& t = g_trace;
    if (on && !t.have_events) {
        for (int i = 0; i <= kMaxTrace; ++i)
            if (cudaEventCreate(&t.ev[i]) != cudaSuccess) return HILS_ERR_CUDA;
        t.have_events = true;
    }
    t.enabled = on != 0;
    t.n = 0;
    return HILS_OK;
}

int hils_trace_read(char* names, size_t names_bytes, float* ms, int max_kernels) {
    Trace& t = g_trace;
    if (!t.enabled || !t.have_events) return 0;
    if (!ms || max_kernels < 0) return HILS_ERR_INVALID_ARG;
    if (t.n > 0 && cudaEventSynchronize(t.ev[t.n]) != cudaSuccess) return HILS_ERR_CUDA;
    size_t off = 0;
    if (names && names_bytes) names[0] = 0;
    int n = t.n < max_kernels ? t.n : max_kernels;
    for (int i = 0; i < n; ++i) {
        if (cudaEventElapsedTime(&ms[i], t.ev[i], t.ev[i + 1]) != cudaSuccess) return HILS_ERR_CUDA;
        if (names) {
            const size_t len = strlen(t.names[i]);
            if (off + len + 2 <= names_bytes) {
                memcpy(names + off, t.names[i], len);
                off += len;
                names[off++] = ';';
                names[off] = 0;
            }
        }
    }
    return n;
}

const char* hils_status_string(int status) {
    switch (status) {
        case HILS_OK: return "ok";
        case HILS_ERR_INVALID_ARG: return "invalid argument";
        case HILS_ERR_UNSUPPORTED: return "unsupported shape or option";
        case HILS_ERR_ALIGNMENT: return "pointer not sufficiently aligned";
        case HILS_ERR_WORKSPACE: return "workspace missing or too small";
        case HILS_ERR_CUDA: return "CUDA runtime error";
        case HILS_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case HILS_ERR_DEVICE_INDEX: return "device-side index out of range";
        default: return "unknown status";
    }
}

const char* hils_version(void) { return "0.1"; }

}  // extern "C"
