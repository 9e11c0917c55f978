// The C ABI of the bounded-cache attention library: argument validation, the opaque
// handle, workspace carve-up and the launch sequence of each entry point.  No device
// memory is allocated here; everything lives in the caller's workspace.
#include <cuda_runtime.h>

#include <mutex>

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <unordered_set>

#include "bct_internal.h"

namespace {

thread_local char g_err[512] = "";

bct_status_t fail(bct_status_t st, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return st;
}

bct_status_t fail_cuda(const char* what, cudaError_t e) {
    return fail(BCT_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Offsets of the workspace sections.
struct Carve {
    size_t kplane, vhi, vlo, status, stage_q[2], stage_k[2], stage_v[2], stage_out[2], total;
    size_t plane_bytes, q_bytes, kv_bytes, out_bytes;  // staging for max_stream tokens
};

bct_status_t resolve_params(const bct_params_t* in, bct_params_t* p) {
    if (in == nullptr) return fail(BCT_ERR_INVALID_ARG, "params is NULL");
    *p = *in;
    if (p->batch < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1 || p->capacity < 1)
        return fail(BCT_ERR_INVALID_ARG, "batch, n_q_heads, n_kv_heads and capacity must be >= 1");
    if (p->n_q_heads % p->n_kv_heads != 0)
        return fail(BCT_ERR_INVALID_ARG, "n_q_heads (%d) is not a multiple of n_kv_heads (%d)", p->n_q_heads,
                    p->n_kv_heads);
    if (p->dtype != BCT_F32 && p->dtype != BCT_BF16) return fail(BCT_ERR_INVALID_ARG, "unknown dtype %d", p->dtype);
    if (p->head_dim < 1) return fail(BCT_ERR_INVALID_ARG, "head_dim must be >= 1");
    if (p->init_len < 0 || p->init_len > p->capacity)
        return fail(BCT_ERR_INVALID_ARG, "init_len %d outside 0..capacity (%d)", p->init_len, p->capacity);
    if (p->flags & ~(BCT_FLAG_SKIP_FIRST_WRITE | BCT_FLAG_WRITE_THEN_READ | BCT_FLAG_DENSE_WRITE | BCT_FLAG_OUT_F32 |
                     BCT_FLAG_PRECISE_READ | BCT_FLAG_CUDA_CORES))
        return fail(BCT_ERR_INVALID_ARG, "unknown flag bits 0x%x", p->flags);
    if (!(p->read_scale > 0.f)) p->read_scale = 1.0f / std::sqrt((float)p->head_dim);
    if (!(p->write_scale > 0.f)) p->write_scale = 1.0f;
    if (!(p->write_eps > 0.f)) p->write_eps = 5.9604644775390625e-08f;  // 2^-24
    if (p->max_stream <= 0) p->max_stream = 1;
    if ((long long)p->batch * p->n_kv_heads > (1LL << 24))
        return fail(BCT_ERR_INVALID_ARG, "batch * n_kv_heads too large");
    if (p->head_dim != 64 && p->head_dim != 128)
        return fail(BCT_ERR_UNSUPPORTED, "head_dim %d: this library has kernels for 64 and 128", p->head_dim);
    if (p->n_q_heads / p->n_kv_heads > bct::kMaxGroupTc)
        return fail(BCT_ERR_UNSUPPORTED, "group size %d > %d", p->n_q_heads / p->n_kv_heads, bct::kMaxGroupTc);
    return BCT_OK;
}

Carve carve(const bct_params_t& p) {
    Carve c;
    const size_t eb = p.dtype == BCT_F32 ? 4 : 2;
    const size_t U = (size_t)p.batch * p.n_kv_heads;
    c.plane_bytes = U * (size_t)p.capacity * p.head_dim * eb;
    c.q_bytes = (size_t)p.batch * p.max_stream * p.n_q_heads * p.head_dim * eb;
    c.kv_bytes = (size_t)p.batch * p.max_stream * p.n_kv_heads * p.head_dim * eb;
    c.out_bytes = (p.flags & BCT_FLAG_OUT_F32) ? c.q_bytes / eb * 4 : c.q_bytes;
    size_t off = 0;
    c.kplane = off;
    off += round_up(c.plane_bytes, bct::kAlign);
    c.vhi = off;
    off += round_up(c.plane_bytes, bct::kAlign);
    c.vlo = off;
    off += (p.dtype == BCT_BF16) ? round_up(c.plane_bytes, bct::kAlign) : 0;
    c.status = off;
    off += bct::kAlign + round_up(U * sizeof(unsigned long long), bct::kAlign);  // status words, then one progress word per unit
    for (int i = 0; i < 2; ++i) {  // two staging sets: one call's copies overlap the previous call's kernel
        c.stage_q[i] = off;
        off += round_up(c.q_bytes, bct::kAlign);
        c.stage_k[i] = off;
        off += round_up(c.kv_bytes, bct::kAlign);
        c.stage_v[i] = off;
        off += round_up(c.kv_bytes, bct::kAlign);
        c.stage_out[i] = off;
        off += round_up(c.out_bytes, bct::kAlign);
    }
    c.total = off;
    return c;
}

// The handles bct_cache_create has given out and bct_cache_destroy has not yet taken back.  A handle
// is looked up here before it is dereferenced, so that a destroyed one is refused, not read.
std::mutex g_live_mu;
std::unordered_set<const bct_cache_t*>& live_handles() {
    static std::unordered_set<const bct_cache_t*> set;
    return set;
}
bool handle_is_live(const bct_cache_t* c) {
    std::lock_guard<std::mutex> lock(g_live_mu);
    return live_handles().count(c) != 0;
}

bct_status_t check_handle(const bct_cache_t* c) {
    if (c == nullptr) return fail(BCT_ERR_INVALID_ARG, "cache handle is NULL");
    if (!handle_is_live(c) || c->magic != bct::kMagic)
        return fail(BCT_ERR_STATE, "cache handle is destroyed or was never created");
    return BCT_OK;
}

bct_status_t check_step_ptrs(const void* q, const void* k, const void* v, const void* out, bool out_optional) {
    if (q == nullptr || k == nullptr || v == nullptr) return fail(BCT_ERR_INVALID_ARG, "q, k and v must not be NULL");
    if (out == nullptr && !out_optional) return fail(BCT_ERR_INVALID_ARG, "out must not be NULL");
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out))
        return fail(BCT_ERR_INVALID_ARG, "q, k, v and out must be 16-byte aligned");
    return BCT_OK;
}

void release_host_objects(bct_cache_t* c) {
    for (int i = 0; i < 2; ++i) {
        if (c->ev_in[i]) cudaEventDestroy(c->ev_in[i]);
        if (c->ev_free[i]) cudaEventDestroy(c->ev_free[i]);
        c->ev_in[i] = c->ev_free[i] = nullptr;
    }
    if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
    c->copy_stream = nullptr;
}

// Tokens [t, T) of the call into a full cache with nothing read: the write-only chunks of the stream
// kernel (128 tokens, then one shorter chunk rounded up to 16 whose rows past T are zero-filled).
bct_status_t write_only_tokens(bct_cache_t* c, const void* k, const void* v, const float* eta, int64_t T, int64_t t,
                               cudaStream_t stream) {
    const int64_t whole = (T - t) / 128, rest = (T - t) - whole * 128;
    cudaError_t e = cudaSuccess;
    if (whole > 0) {
        const int n = bct::launch_stream_tc(c, nullptr, k, v, nullptr, T, eta, t, whole, -1, 1, 128, stream, &e);
        if (n < 0) return fail_cuda("write-only stream launch", e);
        c->launches += n;
    }
    if (rest > 0) {
        const int tc = (int)((rest + 15) / 16 * 16);
        const int n = bct::launch_stream_tc(c, nullptr, k, v, nullptr, T, eta, t + whole * 128, 1, -1, 1, tc, stream, &e);
        if (n < 0) return fail_cuda("write-only stream launch", e);
        c->launches += n;
    }
    c->n_full_tokens += T - t;
    return BCT_OK;
}

// T tokens of the [B][T][H][d] step arrays (device pointers) through the cache: whole chunks on the
// chunked stream kernel where it applies, single tokens on the decode kernels otherwise.  Everything
// that can be refused on the host has been refused by the callers; a failure here is the CUDA runtime
// refusing a launch, and the counters then describe exactly the tokens already enqueued.
// eta: [B][T][Hkv] floats on the device, or NULL.
bct_status_t run_tokens(bct_cache_t* c, const void* q, const void* k, const void* v, const float* eta, void* out,
                        int64_t T, cudaStream_t stream) {
    const bct_params_t& p = c->p;
    const size_t eb = (size_t)c->elem_bytes;
    const size_t q_tok = (size_t)p.n_q_heads * p.head_dim;   // elements per token per sequence
    const size_t kv_tok = (size_t)p.n_kv_heads * p.head_dim;
    const int Tc = bct::stream_chunk_tokens(c);
    int64_t t = 0;
    while (t < T) {
        const bool full = (c->len == p.capacity);
        const int do_write = !((p.flags & BCT_FLAG_SKIP_FIRST_WRITE) && c->n_full_tokens == 0);
        // no output asked for (UpdateKV): the rest of the call goes through the write-only chunks
        if (out == nullptr && Tc > 0 && full && do_write && T - t >= 4) return write_only_tokens(c, k, v, eta, T, t, stream);
        // whole chunks against a full cache go through the chunked tensor-core kernel
        if (Tc > 0 && full && do_write && T - t >= Tc) {
            const int64_t n_chunks = (T - t) / Tc;
            cudaError_t e = cudaSuccess;
            const int n = bct::launch_stream_tc(c, q, k, v, out, T, eta, t, n_chunks, -1, 0, 0, stream, &e);
            if (n < 0) return fail_cuda("stream launch", e);
            c->launches += n;
            c->n_full_tokens += n_chunks * Tc;
            t += n_chunks * Tc;
            continue;
        }
        // whole chunks that still fit the free slots are appended by the same kernel in its fill mode
        if (Tc > 0 && !full && T - t >= Tc && p.capacity - c->len >= Tc) {
            const int64_t by_tokens = (T - t) / Tc, by_slots = (p.capacity - c->len) / Tc;
            const int64_t n_chunks = by_tokens < by_slots ? by_tokens : by_slots;
            cudaError_t e = cudaSuccess;
            const int n = bct::launch_stream_tc(c, q, k, v, out, T, eta, t, n_chunks, c->len, 0, 0, stream, &e);
            if (n < 0) return fail_cuda("stream launch (fill)", e);
            c->launches += n;
            c->len += (int)(n_chunks * Tc);
            t += n_chunks * Tc;
            continue;
        }
        // the ragged end of the call: with a full cache one shorter chunk (rounded up to 8 tokens; the rows past
        // the last token are zero-filled, add nothing and store nothing); while the cache fills, a chunk of
        // exactly the largest multiple of 8 that fits, and single tokens for the rest
        // (a chunk streams the unit's planes about three times as often as a decode step does: not below 4 tokens)
        if (Tc > 0 && full && do_write && T - t >= 4) {
            const int64_t r = T - t;  // < Tc here
            const int tc = (int)((r + 7) / 8 * 8);
            cudaError_t e = cudaSuccess;
            const int n = bct::launch_stream_tc(c, q, k, v, out, T, eta, t, 1, -1, 0, tc, stream, &e);
            if (n < 0) return fail_cuda("stream launch (last chunk)", e);
            c->launches += n;
            c->n_full_tokens += r;
            t += r;
            continue;
        }
        if (Tc > 0 && !full) {
            const int64_t m = T - t < p.capacity - c->len ? T - t : p.capacity - c->len;  // < Tc here
            const int tc = (int)(m / 8 * 8);
            if (tc >= 8) {
                cudaError_t e = cudaSuccess;
                const int n = bct::launch_stream_tc(c, q, k, v, out, T, eta, t, 1, c->len, 0, tc, stream, &e);
                if (n < 0) return fail_cuda("stream launch (fill, last chunk)", e);
                c->launches += n;
                c->len += tc;
                t += tc;
                continue;
            }
        }
        bct::StepIO io;
        io.q = static_cast<const char*>(q) + (size_t)t * q_tok * eb;
        io.k = static_cast<const char*>(k) + (size_t)t * kv_tok * eb;
        io.v = static_cast<const char*>(v) + (size_t)t * kv_tok * eb;
        const size_t ob = (p.flags & BCT_FLAG_OUT_F32) ? 4 : eb;
        io.out = out ? static_cast<char*>(out) + (size_t)t * q_tok * ob : nullptr;
        io.q_batch_stride = (int64_t)(T * q_tok);
        io.kv_batch_stride = (int64_t)(T * kv_tok);
        io.eta = eta ? eta + (size_t)t * p.n_kv_heads : nullptr;
        io.eta_batch_stride = (int64_t)T * p.n_kv_heads;
        cudaError_t e = cudaSuccess;
        const int n = bct::launch_decode(c, io, c->len, do_write, stream, &e);
        if (n < 0) return fail_cuda("decode launch", e);
        c->launches += n;
        if (full)
            c->n_full_tokens += 1;
        else
            c->len += 1;
        ++t;
    }
    return BCT_OK;
}

}  // namespace

namespace bct {
void set_last_error(const char* msg) { snprintf(g_err, sizeof(g_err), "%s", msg); }
bct_status_t check_live_handle(const bct_cache* c) { return check_handle(c); }
}  // namespace bct

extern "C" {

int32_t bct_version(void) { return 100; }

const char* bct_last_error(void) { return g_err; }

bct_status_t bct_cache_bytes(const bct_params_t* params, size_t* bytes, size_t* align) {
    bct_params_t p;
    bct_status_t st = resolve_params(params, &p);
    if (st != BCT_OK) return st;
    if (bytes == nullptr) return fail(BCT_ERR_INVALID_ARG, "bytes is NULL");
    *bytes = carve(p).total;
    if (align) *align = bct::kAlign;
    return BCT_OK;
}

bct_status_t bct_cache_create(const bct_params_t* params, void* workspace, size_t bytes, const void* mk_init,
                              const void* mv_init, void* cuda_stream, bct_cache_t** out) {
    bct_params_t p;
    bct_status_t st = resolve_params(params, &p);
    if (st != BCT_OK) return st;
    if (out == nullptr) return fail(BCT_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (workspace == nullptr) return fail(BCT_ERR_INVALID_ARG, "workspace is NULL");
    if (reinterpret_cast<uintptr_t>(workspace) % bct::kAlign)
        return fail(BCT_ERR_INVALID_ARG, "workspace must be %zu-byte aligned", bct::kAlign);
    const Carve cv = carve(p);
    if (bytes < cv.total) return fail(BCT_ERR_INVALID_ARG, "workspace of %zu bytes, %zu needed", bytes, cv.total);
    if (p.init_len > 0 && mk_init == nullptr) return fail(BCT_ERR_INVALID_ARG, "mk_init is NULL with init_len > 0");
    if (!aligned16(mk_init) || !aligned16(mv_init)) return fail(BCT_ERR_INVALID_ARG, "mk_init / mv_init misaligned");

    int dev = 0, sms = 0, optin = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e != cudaSuccess) return fail_cuda("device query", e);
    const char* why = "";
    const bool tc_only = p.n_q_heads / p.n_kv_heads > bct::kMaxGroup;  // 9..15 query heads per kv-head: tensor-core kernel only
    if (!tc_only && !bct::decode_supported(p, optin, &why)) return fail(BCT_ERR_UNSUPPORTED, "%s", why);

    bct_cache_t* c = new (std::nothrow) bct_cache_t();
    if (c == nullptr) return fail(BCT_ERR_STATE, "out of host memory");
    c->magic = bct::kMagic;
    c->p = p;
    c->G = p.n_q_heads / p.n_kv_heads;
    c->U = p.batch * p.n_kv_heads;
    c->elem_bytes = p.dtype == BCT_F32 ? 4 : 2;
    c->row_bytes = (size_t)p.head_dim * c->elem_bytes;
    c->plane_bytes = cv.plane_bytes;
    c->ws = static_cast<char*>(workspace);
    c->ws_bytes = bytes;
    c->kplane = c->ws + cv.kplane;
    c->vhi = c->ws + cv.vhi;
    c->vlo = p.dtype == BCT_BF16 ? c->ws + cv.vlo : nullptr;
    c->status = reinterpret_cast<int*>(c->ws + cv.status);
    c->progress = reinterpret_cast<unsigned long long*>(c->ws + cv.status + bct::kAlign);
    c->stream_launches = 0;
    for (int i = 0; i < 2; ++i) {
        c->stage_q[i] = c->ws + cv.stage_q[i];
        c->stage_k[i] = c->ws + cv.stage_k[i];
        c->stage_v[i] = c->ws + cv.stage_v[i];
        c->stage_out[i] = c->ws + cv.stage_out[i];
        c->ev_in[i] = nullptr;
        c->ev_free[i] = nullptr;
    }
    c->copy_stream = nullptr;
    c->host_calls = 0;
    c->len = p.init_len;
    c->n_full_tokens = 0;
    c->launches = 0;
    c->device = dev;
    c->sm_count = sms;
    c->smem_optin = optin;

    // a stream and four events of the handle's own (host objects: no device memory)
    e = cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking);
    for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
        e = cudaEventCreateWithFlags(&c->ev_in[i], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_free[i], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) {
        release_host_objects(c);
        c->magic = 0;
        delete c;
        return fail_cuda("stream / event creation", e);
    }
    bct::tc_prepare(c);  // tensor maps of the planes; without them the CUDA-core kernel serves every shape
    if (tc_only && (!bct::tc_eligible(c) || (p.flags & BCT_FLAG_CUDA_CORES))) {
        release_host_objects(c);
        c->magic = 0;
        delete c;
        return fail(BCT_ERR_UNSUPPORTED,
                    "group sizes 9..15 are served by the tensor-core kernel only: bfloat16, head_dim 128, 128 <= capacity "
                    "<= 65536, K plane >= 256 KiB, no PRECISE_READ / CUDA_CORES");
    }

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    e = cudaMemsetAsync(c->status, 0, cv.stage_q[0] - cv.status, stream);  // status and progress words
    if (e == cudaSuccess) e = bct::launch_import(c, mk_init, mv_init, p.dtype, p.init_len, stream);
    if (e != cudaSuccess) {
        release_host_objects(c);
        c->magic = 0;
        delete c;
        return fail_cuda("state import", e);
    }
    c->launches += 1;
    {
        std::lock_guard<std::mutex> lock(g_live_mu);
        live_handles().insert(c);
    }
    *out = c;
    return BCT_OK;
}

bct_status_t bct_decode_step(bct_cache_t* c, const void* q, const void* k, const void* v, void* out,
                             void* cuda_stream) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    st = check_step_ptrs(q, k, v, out, false);
    if (st != BCT_OK) return st;
    return run_tokens(c, q, k, v, nullptr, out, 1, static_cast<cudaStream_t>(cuda_stream));
}

bct_status_t bct_prefill_stream(bct_cache_t* c, const void* q, const void* k, const void* v, void* out, int64_t T,
                                void* cuda_stream) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    if (T < 1 || T > bct::kMaxCallTokens)
        return fail(BCT_ERR_INVALID_ARG, "T must be in [1, 2^30] (got %lld)", (long long)T);
    st = check_step_ptrs(q, k, v, out, true);
    if (st != BCT_OK) return st;
    return run_tokens(c, q, k, v, nullptr, out, T, static_cast<cudaStream_t>(cuda_stream));
}

bct_status_t bct_prefill_stream_eta(bct_cache_t* c, const void* q, const void* k, const void* v, const float* eta,
                                    void* out, int64_t T, void* cuda_stream) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    if (T < 1 || T > bct::kMaxCallTokens)
        return fail(BCT_ERR_INVALID_ARG, "T must be in [1, 2^30] (got %lld)", (long long)T);
    st = check_step_ptrs(q, k, v, out, true);
    if (st != BCT_OK) return st;
    if ((reinterpret_cast<uintptr_t>(eta) & 3u) != 0) return fail(BCT_ERR_INVALID_ARG, "eta must be 4-byte aligned");
    return run_tokens(c, q, k, v, eta, out, T, static_cast<cudaStream_t>(cuda_stream));
}

bct_status_t bct_update_kv(bct_cache_t* c, const void* wq, const void* wv, const float* eta, int64_t T,
                           void* cuda_stream) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    if (T < 1 || T > bct::kMaxCallTokens)
        return fail(BCT_ERR_INVALID_ARG, "T must be in [1, 2^30] (got %lld)", (long long)T);
    if (wq == nullptr || wv == nullptr) return fail(BCT_ERR_INVALID_ARG, "wq and wv must not be NULL");
    if (!aligned16(wq) || !aligned16(wv)) return fail(BCT_ERR_INVALID_ARG, "wq and wv must be 16-byte aligned");
    if ((reinterpret_cast<uintptr_t>(eta) & 3u) != 0) return fail(BCT_ERR_INVALID_ARG, "eta must be 4-byte aligned");
    if (c->len != c->p.capacity)
        return fail(BCT_ERR_STATE, "UpdateKV works on a full-size MV_0: the cache holds %d of %d slots", c->len,
                    c->p.capacity);
    if (bct::stream_chunk_tokens(c) == 0 || (c->p.flags & BCT_FLAG_SKIP_FIRST_WRITE))
        return fail(BCT_ERR_UNSUPPORTED,
                    "the write-only form serves bfloat16 caches with head_dim 128 and 128..16384 slots, without "
                    "SKIP_FIRST_WRITE; use bct_prefill_stream with out = NULL");
    return write_only_tokens(c, wq, wv, eta, T, 0, static_cast<cudaStream_t>(cuda_stream));
}

bct_status_t bct_update_kv_backward(bct_cache_t* c, const void* wq, const void* wv, const float* eta, const void* d_mv,
                                    int64_t T, float* d_wq, float* d_wv, float* d_mk, float* d_eta, void* cuda_stream) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    if (T < 1 || T > bct::kMaxCallTokens)
        return fail(BCT_ERR_INVALID_ARG, "T must be in [1, 2^30] (got %lld)", (long long)T);
    if (!wq || !wv || !d_mv || !d_wq || !d_wv) return fail(BCT_ERR_INVALID_ARG, "wq, wv, d_mv, d_wq and d_wv must not be NULL");
    if (!aligned16(wq) || !aligned16(wv) || !aligned16(d_mv) || !aligned16(d_wq) || !aligned16(d_wv) || !aligned16(d_mk))
        return fail(BCT_ERR_INVALID_ARG, "wq, wv, d_mv, d_wq, d_wv and d_mk must be 16-byte aligned");
    if ((reinterpret_cast<uintptr_t>(eta) & 3u) != 0 || (reinterpret_cast<uintptr_t>(d_eta) & 3u) != 0)
        return fail(BCT_ERR_INVALID_ARG, "eta and d_eta must be 4-byte aligned");
    if (c->len != c->p.capacity)
        return fail(BCT_ERR_STATE, "UpdateKV works on a full-size cache: this one holds %d of %d slots", c->len,
                    c->p.capacity);
    if (!bct::update_bwd_supported(c))
        return fail(BCT_ERR_UNSUPPORTED, "the backward serves bfloat16 caches with head_dim 128 and 128..16384 slots");
    cudaError_t e = cudaSuccess;
    const int n = bct::launch_update_bwd(c, wq, wv, eta, d_mv, T, d_wq, d_wv, d_mk, d_eta,
                                         static_cast<cudaStream_t>(cuda_stream), &e);
    if (n < 0) return fail_cuda("UpdateKV backward launch", e);
    c->launches += n;
    return BCT_OK;
}

bct_status_t bct_decode_step_eta(bct_cache_t* c, const void* q, const void* k, const void* v, const float* eta,
                                 void* out, void* cuda_stream) {
    if (out == nullptr) return fail(BCT_ERR_INVALID_ARG, "out must not be NULL");
    return bct_prefill_stream_eta(c, q, k, v, eta, out, 1, cuda_stream);
}

namespace {

bct_status_t check_project_args(int64_t n_tokens, int32_t d_model, int32_t n_q, int32_t n_kv, const void* x,
                                const void* w_q, const void* w_wq, const void* w_wv, const void* q, const void* k,
                                const void* v) {
    if (n_tokens < 1 || n_tokens > ((int64_t)1 << 31) - 256)
        return fail(BCT_ERR_INVALID_ARG, "n_tokens must be in [1, 2^31 - 256] (got %lld)", (long long)n_tokens);
    if (d_model < 8 || d_model % 8 != 0)
        return fail(BCT_ERR_INVALID_ARG, "d_model must be a positive multiple of 8 (got %d)", d_model);
    if (n_q < 32 || n_q % 32 != 0 || n_kv < 32 || n_kv % 32 != 0)
        return fail(BCT_ERR_UNSUPPORTED, "output features must be positive multiples of 32 (got %d and %d)", n_q, n_kv);
    if (!x || !w_q || !w_wq || !w_wv || !q || !k || !v) return fail(BCT_ERR_INVALID_ARG, "no pointer may be NULL");
    if (!aligned16(x) || !aligned16(w_q) || !aligned16(w_wq) || !aligned16(w_wv) || !aligned16(q) || !aligned16(k) ||
        !aligned16(v))
        return fail(BCT_ERR_INVALID_ARG, "every pointer must be 16-byte aligned");
    return BCT_OK;
}

// SM count and opt-in shared memory of the current device, which must offer the sm_100 tensor path.
// Looked up once per device: the projection of a decode step takes tens of microseconds, and four
// attribute queries per call were a visible part of it.
bct_status_t tensor_device(int* device, int* sm_count, int* smem_optin) {
    constexpr int kMaxDev = 64;
    static std::mutex mu;
    static int known[kMaxDev] = {}, sms[kMaxDev] = {}, optin[kMaxDev] = {}, majors[kMaxDev] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail_cuda("device query", e);
    if (dev < 0 || dev >= kMaxDev) return fail(BCT_ERR_UNSUPPORTED, "device index %d out of range", dev);
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!known[dev]) {
            e = cudaDeviceGetAttribute(&majors[dev], cudaDevAttrComputeCapabilityMajor, dev);
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev);
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin[dev], cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
            if (e != cudaSuccess) return fail_cuda("device query", e);
            known[dev] = 1;
        }
        *device = dev;
        *sm_count = sms[dev];
        *smem_optin = optin[dev];
        if (majors[dev] != 10) return fail(BCT_ERR_UNSUPPORTED, "the projections need an sm_100 device");
    }
    return BCT_OK;
}

inline size_t round256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

bct_status_t bct_project_qkv(int64_t n_tokens, int32_t d_model, int32_t n_q, int32_t n_kv, const void* x,
                             const void* w_q, const void* w_wq, const void* w_wv, void* q, void* k, void* v,
                             void* cuda_stream) {
    bct_status_t st = check_project_args(n_tokens, d_model, n_q, n_kv, x, w_q, w_wq, w_wv, q, k, v);
    if (st != BCT_OK) return st;
    int device = 0, sm_count = 0, smem_optin = 0;
    st = tensor_device(&device, &sm_count, &smem_optin);
    if (st != BCT_OK) return st;
    cudaError_t e = bct::launch_project(n_tokens, d_model, n_q, n_kv, x, w_q, w_wq, w_wv, q, k, v, nullptr, device, sm_count,
                                        smem_optin, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return fail_cuda("projection launch", e);
    return BCT_OK;
}

bct_status_t bct_layer_scratch_bytes(const bct_cache_t* c, int64_t T, size_t* bytes) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    if (T < 1 || T > bct::kMaxCallTokens || bytes == nullptr)
        return fail(BCT_ERR_INVALID_ARG, "T must be in [1, 2^30] and bytes not NULL");
    const size_t eb = (size_t)c->elem_bytes;
    const size_t qb = (size_t)c->p.batch * (size_t)T * c->p.n_q_heads * c->p.head_dim * eb;
    const size_t kb = (size_t)c->p.batch * (size_t)T * c->p.n_kv_heads * c->p.head_dim * eb;
    *bytes = round256(qb) + 2 * round256(kb);
    return BCT_OK;
}

bct_status_t bct_layer_forward(bct_cache_t* c, const void* x, const void* w_q, const void* w_wq, const void* w_wv,
                               int32_t d_model, const float* eta, void* scratch, size_t scratch_bytes, void* out,
                               int64_t T, void* cuda_stream) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    if (c->p.dtype != BCT_BF16) return fail(BCT_ERR_UNSUPPORTED, "the fused projections serve bfloat16 caches only");
    if (T < 1 || T > bct::kMaxCallTokens)
        return fail(BCT_ERR_INVALID_ARG, "T must be in [1, 2^30] (got %lld)", (long long)T);
    size_t need = 0;
    st = bct_layer_scratch_bytes(c, T, &need);
    if (st != BCT_OK) return st;
    if (scratch == nullptr || scratch_bytes < need || (reinterpret_cast<uintptr_t>(scratch) & 255u) != 0)
        return fail(BCT_ERR_INVALID_ARG, "scratch must be 256-byte aligned and hold %zu bytes (got %zu)", need,
                    scratch_bytes);
    const bct_params_t& p = c->p;
    const int n_q = p.n_q_heads * p.head_dim, n_kv = p.n_kv_heads * p.head_dim;
    const int64_t n_tokens = (int64_t)p.batch * T;
    const size_t qb = round256((size_t)n_tokens * n_q * 2), kb = round256((size_t)n_tokens * n_kv * 2);
    char* q = static_cast<char*>(scratch);
    char* k = q + qb;
    char* v = k + kb;
    st = check_project_args(n_tokens, d_model, n_q, n_kv, x, w_q, w_wq, w_wv, q, k, v);
    if (st != BCT_OK) return st;
    if (out != nullptr && !aligned16(out)) return fail(BCT_ERR_INVALID_ARG, "out must be 16-byte aligned");
    if ((reinterpret_cast<uintptr_t>(eta) & 3u) != 0) return fail(BCT_ERR_INVALID_ARG, "eta must be 4-byte aligned");
    if (!c->tc_ready) return fail(BCT_ERR_UNSUPPORTED, "the projections need the driver's tensor-map encoder");
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = bct::launch_project(n_tokens, d_model, n_q, n_kv, x, w_q, w_wq, w_wv, q, k, v, c->status,
                                        c->device, c->sm_count, c->smem_optin, stream);
    if (e != cudaSuccess) return fail_cuda("projection launch", e);
    c->launches += 1;
    return run_tokens(c, q, k, v, eta, out, T, stream);
}

namespace {

// Validation shared by the two stack calls; fills the per-layer scratch need and the activation size.
bct_status_t stack_plan(bct_cache_t* const* caches, int32_t n_layers, int64_t T, size_t* layer_scratch, size_t* act_bytes) {
    if (caches == nullptr || n_layers < 1 || n_layers > 1024)
        return fail(BCT_ERR_INVALID_ARG, "caches must not be NULL and n_layers must be in [1, 1024]");
    if (T < 1 || T > bct::kMaxCallTokens) return fail(BCT_ERR_INVALID_ARG, "T must be in [1, 2^30] (got %lld)", (long long)T);
    *layer_scratch = 0;
    *act_bytes = 0;
    for (int l = 0; l < n_layers; ++l) {
        bct_status_t st = check_handle(caches[l]);
        if (st != BCT_OK) return st;
        const bct_params_t& p = caches[l]->p;
        if (p.dtype != BCT_BF16 || (p.flags & BCT_FLAG_OUT_F32))
            return fail(BCT_ERR_UNSUPPORTED, "layer %d: a stack needs bfloat16 caches with bfloat16 outputs", l);
        if (p.batch != caches[0]->p.batch) return fail(BCT_ERR_INVALID_ARG, "layer %d: batch differs from layer 0", l);
        for (int k = 0; k < l; ++k)
            if (caches[k] == caches[l]) return fail(BCT_ERR_INVALID_ARG, "layer %d: the same cache twice", l);
        size_t need = 0;
        st = bct_layer_scratch_bytes(caches[l], T, &need);
        if (st != BCT_OK) return st;
        if (need > *layer_scratch) *layer_scratch = need;
        const size_t act = round256((size_t)p.batch * (size_t)T * p.n_q_heads * p.head_dim * 2);
        if (l + 1 < n_layers && act > *act_bytes) *act_bytes = act;
    }
    return BCT_OK;
}

}  // namespace

bct_status_t bct_stack_scratch_bytes(bct_cache_t* const* caches, int32_t n_layers, int64_t T, size_t* bytes) {
    if (bytes == nullptr) return fail(BCT_ERR_INVALID_ARG, "bytes is NULL");
    size_t layer_scratch = 0, act = 0;
    bct_status_t st = stack_plan(caches, n_layers, T, &layer_scratch, &act);
    if (st != BCT_OK) return st;
    *bytes = layer_scratch + 2 * act;
    return BCT_OK;
}

bct_status_t bct_stack_forward(bct_cache_t* const* caches, int32_t n_layers, const void* x, int32_t d_model,
                               const void* const* w_q, const void* const* w_wq, const void* const* w_wv, void* scratch,
                               size_t scratch_bytes, void* out, int64_t T, void* cuda_stream) {
    size_t layer_scratch = 0, act = 0;
    bct_status_t st = stack_plan(caches, n_layers, T, &layer_scratch, &act);
    if (st != BCT_OK) return st;
    if (x == nullptr || out == nullptr || w_q == nullptr || w_wq == nullptr || w_wv == nullptr)
        return fail(BCT_ERR_INVALID_ARG, "x, out and the weight arrays must not be NULL");
    if (scratch == nullptr || (reinterpret_cast<uintptr_t>(scratch) & 255u) != 0 || scratch_bytes < layer_scratch + 2 * act)
        return fail(BCT_ERR_INVALID_ARG, "scratch must be 256-byte aligned and hold %zu bytes (got %zu)",
                    layer_scratch + 2 * act, scratch_bytes);
    // everything the layers would refuse is refused here, before the first of them is enqueued
    int dm = d_model;
    for (int l = 0; l < n_layers; ++l) {
        const bct_params_t& p = caches[l]->p;
        const int n_q = p.n_q_heads * p.head_dim, n_kv = p.n_kv_heads * p.head_dim;
        st = check_project_args((int64_t)p.batch * T, dm, n_q, n_kv, x, w_q[l], w_wq[l], w_wv[l], scratch, scratch, scratch);
        if (st != BCT_OK) return st;
        if (!caches[l]->tc_ready) return fail(BCT_ERR_UNSUPPORTED, "layer %d: the projections need the driver's tensor-map encoder", l);
        dm = n_q;
    }
    if (!aligned16(out)) return fail(BCT_ERR_INVALID_ARG, "out must be 16-byte aligned");
    char* base = static_cast<char*>(scratch);
    char* acts[2] = {base + layer_scratch, base + layer_scratch + act};
    const void* in = x;
    dm = d_model;
    for (int l = 0; l < n_layers; ++l) {
        void* o = (l + 1 == n_layers) ? out : static_cast<void*>(acts[l & 1]);
        st = bct_layer_forward(caches[l], in, w_q[l], w_wq[l], w_wv[l], dm, nullptr, base, layer_scratch, o, T, cuda_stream);
        if (st != BCT_OK) return st;
        in = o;
        dm = caches[l]->p.n_q_heads * caches[l]->p.head_dim;
    }
    return BCT_OK;
}

bct_status_t bct_prefill_stream_host(bct_cache_t* c, const void* q, const void* k, const void* v, void* out,
                                     int64_t T, void* cuda_stream) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    if (T < 1) return fail(BCT_ERR_INVALID_ARG, "T must be >= 1 (got %lld)", (long long)T);
    if (T > c->p.max_stream)
        return fail(BCT_ERR_INVALID_ARG, "T = %lld exceeds max_stream = %d given at create", (long long)T,
                    c->p.max_stream);
    if (q == nullptr || k == nullptr || v == nullptr) return fail(BCT_ERR_INVALID_ARG, "q, k and v must not be NULL");
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t eb = (size_t)c->elem_bytes;
    const size_t qb = (size_t)c->p.batch * T * c->p.n_q_heads * c->p.head_dim * eb;
    const size_t kb = (size_t)c->p.batch * T * c->p.n_kv_heads * c->p.head_dim * eb;
    // The inputs go up on the handle's copy stream into the staging set that is not in use, so that
    // they overlap the previous call's kernel; the step itself and the copy of `out` run on `stream`.
    const int set = (int)(c->host_calls & 1);
    cudaError_t e = cudaStreamWaitEvent(c->copy_stream, c->ev_free[set], 0);  // the set's last user is done
    if (e == cudaSuccess) e = cudaMemcpyAsync(c->stage_q[set], q, qb, cudaMemcpyHostToDevice, c->copy_stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(c->stage_k[set], k, kb, cudaMemcpyHostToDevice, c->copy_stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(c->stage_v[set], v, kb, cudaMemcpyHostToDevice, c->copy_stream);
    if (e == cudaSuccess) e = cudaEventRecord(c->ev_in[set], c->copy_stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, c->ev_in[set], 0);
    if (e != cudaSuccess) return fail_cuda("host-to-device copy", e);
    c->host_calls += 1;
    st = run_tokens(c, c->stage_q[set], c->stage_k[set], c->stage_v[set], nullptr, out ? c->stage_out[set] : nullptr, T,
                    stream);
    if (st != BCT_OK) return st;
    if (out != nullptr) {
        const size_t ob = (c->p.flags & BCT_FLAG_OUT_F32) ? qb / eb * 4 : qb;
        e = cudaMemcpyAsync(out, c->stage_out[set], ob, cudaMemcpyDeviceToHost, stream);
        if (e != cudaSuccess) return fail_cuda("device-to-host copy", e);
    }
    e = cudaEventRecord(c->ev_free[set], stream);
    if (e != cudaSuccess) return fail_cuda("event record", e);
    return BCT_OK;
}

bct_status_t bct_decode_step_host(bct_cache_t* c, const void* q, const void* k, const void* v, void* out,
                                  void* cuda_stream) {
    if (out == nullptr) return fail(BCT_ERR_INVALID_ARG, "out must not be NULL");
    return bct_prefill_stream_host(c, q, k, v, out, 1, cuda_stream);
}

bct_status_t bct_cache_len(const bct_cache_t* c, int32_t* len) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    if (len == nullptr) return fail(BCT_ERR_INVALID_ARG, "len is NULL");
    *len = c->len;
    return BCT_OK;
}

bct_status_t bct_cache_export(bct_cache_t* c, void* k_out, void* v_out, int32_t v_dtype, void* cuda_stream) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    if (v_dtype != BCT_F32 && v_dtype != BCT_BF16 && v_dtype != BCT_BF16_PAIR)
        return fail(BCT_ERR_INVALID_ARG, "unknown v_dtype %d", v_dtype);
    if (c->p.dtype == BCT_F32 && v_dtype != BCT_F32)
        return fail(BCT_ERR_UNSUPPORTED, "a float cache exports its values as float");
    if (!aligned16(k_out) || !aligned16(v_out)) return fail(BCT_ERR_INVALID_ARG, "k_out / v_out misaligned");
    if (k_out == nullptr && v_out == nullptr) return BCT_OK;
    cudaError_t e = bct::launch_export(c, k_out, v_out, v_dtype, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return fail_cuda("state export", e);
    c->launches += 1;
    return BCT_OK;
}

bct_status_t bct_cache_import(bct_cache_t* c, const void* k_in, const void* v_in, int32_t v_dtype, int32_t len,
                              void* cuda_stream) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    if (len < 0 || len > c->p.capacity) return fail(BCT_ERR_INVALID_ARG, "len %d outside 0..capacity", len);
    if (v_dtype != BCT_F32 && v_dtype != BCT_BF16 && v_dtype != BCT_BF16_PAIR)
        return fail(BCT_ERR_INVALID_ARG, "unknown v_dtype %d", v_dtype);
    if (c->p.dtype == BCT_F32 && v_dtype != BCT_F32)
        return fail(BCT_ERR_UNSUPPORTED, "a float cache imports its values as float");
    if (len > 0 && k_in == nullptr) return fail(BCT_ERR_INVALID_ARG, "k_in is NULL with len > 0");
    if (!aligned16(k_in) || !aligned16(v_in)) return fail(BCT_ERR_INVALID_ARG, "k_in / v_in misaligned");
    cudaError_t e = bct::launch_import(c, k_in, v_in, v_dtype, len, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return fail_cuda("state import", e);
    c->len = len;
    c->launches += 1;
    return BCT_OK;
}

bct_status_t bct_cache_status(bct_cache_t* c, void* cuda_stream) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int host[2] = {0, 0};
    cudaError_t e = cudaMemcpyAsync(host, c->status, sizeof(host), cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return fail_cuda("status read", e);
    if (host[0] == BCT_ERR_TIMEOUT)
        return fail(BCT_ERR_TIMEOUT, "a bounded wait inside a kernel gave up (site %d)", host[1]);
    if (host[0] != 0) return fail(BCT_ERR_STATE, "device status word holds %d", host[0]);
    return BCT_OK;
}

bct_status_t bct_cache_status_clear(bct_cache_t* c, void* cuda_stream) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    cudaError_t e = cudaMemsetAsync(c->status, 0, 2 * sizeof(int), static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return fail_cuda("status clear", e);
    return BCT_OK;
}

bct_status_t bct_cache_rows_rewritten(bct_cache_t* c, void* cuda_stream, uint64_t* rows) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    if (rows == nullptr) return fail(BCT_ERR_INVALID_ARG, "rows is NULL");
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    unsigned long long host = 0;
    cudaError_t e = cudaMemcpyAsync(&host, c->status + bct::kStatusRowsWord, sizeof(host), cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return fail_cuda("counter read", e);
    *rows = (uint64_t)host;
    return BCT_OK;
}

bct_status_t bct_selftest_timeout(bct_cache_t* c, void* cuda_stream) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    cudaError_t e = bct::launch_wait_selftest(c, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return fail_cuda("self-test launch", e);
    c->launches += 1;
    return BCT_OK;
}

bct_status_t bct_cache_tensor_path(const bct_cache_t* c, int32_t* yes) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    if (yes == nullptr) return fail(BCT_ERR_INVALID_ARG, "yes is NULL");
    *yes = (!(c->p.flags & BCT_FLAG_CUDA_CORES) && bct::tc_eligible(c)) ? 1 : 0;
    return BCT_OK;
}

bct_status_t bct_cache_launches(const bct_cache_t* c, int64_t* launches) {
    bct_status_t st = check_handle(c);
    if (st != BCT_OK) return st;
    if (launches == nullptr) return fail(BCT_ERR_INVALID_ARG, "launches is NULL");
    *launches = c->launches;
    return BCT_OK;
}

bct_status_t bct_cache_destroy(bct_cache_t* c) {
    if (c == nullptr) return BCT_OK;
    {
        std::lock_guard<std::mutex> lock(g_live_mu);
        if (live_handles().erase(c) == 0) return fail(BCT_ERR_STATE, "cache handle is destroyed or was never created");
    }
    release_host_objects(c);
    c->magic = 0;
    delete c;
    return BCT_OK;
}

}  // extern "C"
