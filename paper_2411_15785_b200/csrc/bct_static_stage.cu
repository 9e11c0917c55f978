// bct_prefill_stream_host_static: the host-buffer stream call for callers that cannot allocate.
//
// bct_prefill_stream_host stages the step vectors in the cache's workspace, whose staging area
// was sized once, by max_stream, when the caller allocated the workspace.  A caller that has
// since lost the ability to allocate device memory cannot grow it: a serving loop that runs
// inside a frozen memory pool, a plug-in that is handed a fixed arena by its host application
// and is forbidden to call cudaMalloc, code that runs while another library holds all of the
// device's memory.  For those callers this file keeps a staging area of its own, a file-scope
// __device__ array of kStaticStageBytes that every GPU loading the library holds until the
// process exits, and feeds the ordinary device entry point from it.  Nothing here allocates.
#include <cuda_runtime.h>

#include <cstdio>
#include <mutex>

#include "bct_internal.h"

namespace {

constexpr size_t kStaticStageBytes = BCT_STATIC_STAGE_BYTES;  // 8 MiB per GPU: q, k, v and out of one call
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for the runtime, never an
// address to hand to a kernel or a copy: stage_base() asks the runtime for the device address.
static __device__ __align__(256) unsigned char g_static_stage[kStaticStageBytes];

std::mutex g_mu;
unsigned char* g_base[kMaxDevices] = {};  // device address of g_static_stage on each device

// Device address of the array on `device`, which must be the current device.  Looked up once
// per device (the first call on that device); later calls reuse the pointer.
cudaError_t stage_base(int device, unsigned char** base) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_base[device] == nullptr) {
        unsigned char* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_stage);
        if (e != cudaSuccess) return e;
        g_base[device] = p;
    }
    *base = g_base[device];
    return cudaSuccess;
}

inline size_t round256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

extern "C" {

bct_status_t bct_prefill_stream_host_static(bct_cache_t* c, const void* q, const void* k, const void* v, void* out,
                                            int64_t T, void* cuda_stream) {
    char msg[256] = "";
    bct_status_t hs = bct::check_live_handle(c);
    if (hs != BCT_OK) return hs;
    if (q == nullptr || k == nullptr || v == nullptr || out == nullptr) {
        bct::set_last_error("q, k, v and out must not be NULL");
        return BCT_ERR_INVALID_ARG;
    }
    if (T < 1) {
        snprintf(msg, sizeof(msg), "T must be >= 1 (got %lld)", (long long)T);
        bct::set_last_error(msg);
        return BCT_ERR_INVALID_ARG;
    }
    const bct_params_t& p = c->p;
    const size_t eb = (size_t)c->elem_bytes;
    const size_t ob = (p.flags & BCT_FLAG_OUT_F32) ? 4 : eb;
    // T is bounded before any product with it: the bytes one token of every sequence needs, then the
    // largest T that could fit at all (a huge T must not wrap the sizes below)
    const size_t q_tok = (size_t)p.batch * p.n_q_heads * p.head_dim, kv_tok = (size_t)p.batch * p.n_kv_heads * p.head_dim;
    const size_t per_token = q_tok * (eb + ob) + 2 * kv_tok * eb;
    const bool t_fits = (uint64_t)T <= kStaticStageBytes / per_token;
    const size_t q_elems = t_fits ? q_tok * (size_t)T : 0;
    const size_t kv_elems = t_fits ? kv_tok * (size_t)T : 0;
    const size_t q_bytes = q_elems * eb, kv_bytes = kv_elems * eb, out_bytes = q_elems * ob;
    const size_t need = t_fits ? round256(q_bytes) + 2 * round256(kv_bytes) + round256(out_bytes)
                               : (T > (1 << 20) ? ~(size_t)0 : per_token * (size_t)T);
    if (!t_fits || need > kStaticStageBytes) {
        snprintf(msg, sizeof(msg),
                 "T = %lld needs %zu bytes of staging; the static staging area holds %zu (use fewer tokens per call)",
                 (long long)T, need, kStaticStageBytes);
        bct::set_last_error(msg);
        return BCT_ERR_INVALID_ARG;
    }
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices || dev != c->device) {
        snprintf(msg, sizeof(msg), "the cache's device (%d) must be the current device (%d)", c->device, dev);
        bct::set_last_error(msg);
        return e != cudaSuccess ? BCT_ERR_CUDA : BCT_ERR_INVALID_ARG;
    }
    unsigned char* base = nullptr;
    e = stage_base(dev, &base);
    if (e != cudaSuccess) {
        snprintf(msg, sizeof(msg), "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        bct::set_last_error(msg);
        return BCT_ERR_CUDA;
    }
    unsigned char* dq = base;
    unsigned char* dk = dq + round256(q_bytes);
    unsigned char* dv = dk + round256(kv_bytes);
    unsigned char* dout = dv + round256(kv_bytes);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // Every byte the step reads (q, k, v) is overwritten by these copies and every byte copied
    // back (out) is written by the step, so nothing of the previous call's contents is used and
    // nothing needs clearing.
    e = cudaMemcpyAsync(dq, q, q_bytes, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dk, k, kv_bytes, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dv, v, kv_bytes, cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) {
        snprintf(msg, sizeof(msg), "host-to-device copy: %s", cudaGetErrorString(e));
        bct::set_last_error(msg);
        return BCT_ERR_CUDA;
    }
    bct_status_t st = bct_prefill_stream(c, dq, dk, dv, dout, T, cuda_stream);
    if (st != BCT_OK) return st;  // bct_last_error() already holds the reason
    e = cudaMemcpyAsync(out, dout, out_bytes, cudaMemcpyDeviceToHost, stream);
    if (e != cudaSuccess) {
        snprintf(msg, sizeof(msg), "device-to-host copy: %s", cudaGetErrorString(e));
        bct::set_last_error(msg);
        return BCT_ERR_CUDA;
    }
    return BCT_OK;
}

}  // extern "C"
