// Import and export of the cache state (MK, MV) between the caller's canonical
// [B][Hkv][rows][d] tensors and the workspace planes.  Not on the hot path: plain
// grid-stride element kernels.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "bct_device.cuh"
#include "bct_internal.h"

namespace bct {
namespace {

template <typename T>
__device__ __forceinline__ float load_as_float(const void* p, size_t i) {
    return (float)reinterpret_cast<const T*>(p)[i];
}

// One thread per element of the [U][C][d] planes.
template <typename CacheT>
__global__ void import_kernel(CacheT* kplane, CacheT* vhi, __nv_bfloat16* vlo, const CacheT* k_in,
                              const void* v_in, int v_mode, size_t U, int C, int d, int len) {
    const size_t n = U * (size_t)C * d;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const size_t e = i % d;
        const size_t j = (i / d) % C;
        const size_t u = i / ((size_t)C * d);
        CacheT kk = (CacheT)0.f;
        float vv = 0.f;
        uint32_t pair = 0;
        if ((int)j < len) {
            const size_t src = (u * len + j) * d + e;
            kk = k_in[src];
            if (v_in != nullptr) {
                if (v_mode == 2)
                    pair = reinterpret_cast<const uint32_t*>(v_in)[src];
                else
                    vv = v_mode == 1 ? load_as_float<float>(v_in, src) : load_as_float<CacheT>(v_in, src);
            }
        }
        kplane[i] = kk;
        if (v_mode == 2) {  // bfloat16 cache only: both planes bit for bit
            reinterpret_cast<uint16_t*>(vhi)[i] = (uint16_t)(pair >> 16);
            reinterpret_cast<uint16_t*>(vlo)[i] = (uint16_t)(pair & 0xffffu);
        } else {
            const CacheT hi = (CacheT)vv;
            vhi[i] = hi;
            if (vlo != nullptr) vlo[i] = __float2bfloat16_rn(vv - (float)hi);
        }
    }
}

template <typename CacheT>
__global__ void export_kernel(const CacheT* kplane, const CacheT* vhi, const __nv_bfloat16* vlo, CacheT* k_out,
                              void* v_out, int v_mode, size_t U, int C, int d, int len) {
    const size_t n = U * (size_t)C * d;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const size_t j = (i / d) % C;
        const bool live = (int)j < len;
        if (k_out != nullptr) k_out[i] = live ? kplane[i] : (CacheT)0.f;
        if (v_out != nullptr && v_mode == 2) {
            uint32_t pair = 0;
            if (live)
                pair = ((uint32_t) reinterpret_cast<const uint16_t*>(vhi)[i] << 16) |
                       reinterpret_cast<const uint16_t*>(vlo)[i];
            reinterpret_cast<uint32_t*>(v_out)[i] = pair;
        } else if (v_out != nullptr) {
            const bool v_is_f32 = (v_mode == 1);
            float vv = 0.f;
            if (live) {
                vv = (float)vhi[i];
                if (vlo != nullptr && v_is_f32) vv += __bfloat162float(vlo[i]);  // exact: <= 17 significant bits
            }
            if (v_is_f32)
                reinterpret_cast<float*>(v_out)[i] = vv;
            else
                reinterpret_cast<CacheT*>(v_out)[i] = (CacheT)vv;
        }
    }
}

// Self-test of the bounded waits: a barrier that expects one arrival and never gets it.  The wait
// runs out after `limit` polls, the failure goes to the status words like any other, and the block
// returns normally.
__global__ void wait_selftest_kernel(int* status, uint32_t limit, int site) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_mbar_init_cluster();
        if (!mbar_wait(&bar, 0, limit)) report_timeout(status, site);
    }
}

inline unsigned grid_for(size_t n, int sm_count) {
    size_t blocks = (n + 255) / 256;
    size_t cap = (size_t)sm_count * 16;
    return (unsigned)(blocks < cap ? (blocks ? blocks : 1) : cap);
}

}  // namespace

cudaError_t launch_import(const bct_cache* c, const void* k_in, const void* v_in, int v_dtype, int len,
                          cudaStream_t stream) {
    const size_t n = (size_t)c->U * c->p.capacity * c->p.head_dim;
    const unsigned grid = grid_for(n, c->sm_count);
    const int v_mode = (v_dtype == BCT_F32) ? 1 : (v_dtype == BCT_BF16_PAIR ? 2 : 0);
    if (c->p.dtype == BCT_F32) {
        import_kernel<float><<<grid, 256, 0, stream>>>(reinterpret_cast<float*>(c->kplane), reinterpret_cast<float*>(c->vhi),
                                                       nullptr, static_cast<const float*>(k_in), v_in, 1, (size_t)c->U,
                                                       c->p.capacity, c->p.head_dim, len);
    } else {
        import_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(
            reinterpret_cast<__nv_bfloat16*>(c->kplane), reinterpret_cast<__nv_bfloat16*>(c->vhi),
            reinterpret_cast<__nv_bfloat16*>(c->vlo), static_cast<const __nv_bfloat16*>(k_in), v_in, v_mode,
            (size_t)c->U, c->p.capacity, c->p.head_dim, len);
    }
    return cudaGetLastError();
}

cudaError_t launch_wait_selftest(const bct_cache* c, cudaStream_t stream) {
    wait_selftest_kernel<<<1, 32, 0, stream>>>(c->status, 1000u, 99);
    return cudaGetLastError();
}

cudaError_t launch_export(const bct_cache* c, void* k_out, void* v_out, int v_dtype, cudaStream_t stream) {
    const size_t n = (size_t)c->U * c->p.capacity * c->p.head_dim;
    const unsigned grid = grid_for(n, c->sm_count);
    const int v_mode = (v_dtype == BCT_F32) ? 1 : (v_dtype == BCT_BF16_PAIR ? 2 : 0);
    if (c->p.dtype == BCT_F32) {
        export_kernel<float><<<grid, 256, 0, stream>>>(reinterpret_cast<const float*>(c->kplane),
                                                       reinterpret_cast<const float*>(c->vhi), nullptr,
                                                       static_cast<float*>(k_out), v_out, 1, (size_t)c->U,
                                                       c->p.capacity, c->p.head_dim, c->len);
    } else {
        export_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(
            reinterpret_cast<const __nv_bfloat16*>(c->kplane), reinterpret_cast<const __nv_bfloat16*>(c->vhi),
            reinterpret_cast<const __nv_bfloat16*>(c->vlo), static_cast<__nv_bfloat16*>(k_out), v_out, v_mode,
            (size_t)c->U, c->p.capacity, c->p.head_dim, c->len);
    }
    return cudaGetLastError();
}

}  // namespace bct
