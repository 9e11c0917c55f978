// Host-side internals of the bounded-cache attention library (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/bct.h"

namespace bct {

constexpr uint64_t kMagic = 0x4243545f43414348ull;  // "BCT_CACH"
constexpr size_t kAlign = 256;                      // alignment of every workspace section
constexpr int kMaxGroup = 8;     // query heads per kv-head on the CUDA-core kernel
constexpr int64_t kMaxCallTokens = (int64_t)1 << 30;  // tokens per sequence one call may pass
constexpr int kMaxGroupTc = 15;  // ... on the tensor-core decode kernel (16 operand rows: the read heads + the write query)

// Where the step vectors of one launch live and how to walk them.
struct StepIO {
    const void* q;   // read queries
    const void* k;   // write queries
    const void* v;   // write key-value vectors
    void* out;       // may be NULL in state-only streams
    int64_t q_batch_stride;   // elements between sequences in q / out
    int64_t kv_batch_stride;  // elements between sequences in k / v
    const float* eta = nullptr;     // step size of the write per (sequence, kv-head), or NULL (all ones)
    int64_t eta_batch_stride = 0;   // elements between sequences in eta
};

}  // namespace bct

struct bct_cache {
    uint64_t magic;
    bct_params_t p;  // scales, eps and max_stream resolved to their effective values
    int G;           // query heads per kv-head
    int U;           // units = batch * n_kv_heads
    int elem_bytes;
    size_t row_bytes;    // head_dim * elem_bytes
    size_t plane_bytes;  // U * capacity * row_bytes
    char* ws;
    size_t ws_bytes;
    char* kplane;   // MK  [U][C][d]
    char* vhi;      // MV  [U][C][d] (value, or its bfloat16 head)
    char* vlo;      // MV residual plane (bfloat16 only), else NULL
    int* status;    // device status words
    unsigned long long* progress;  // [U] (launch number << 32 | chunks done) of the chunked stream kernel, behind the status words
    mutable uint32_t stream_launches;  // launches of the chunked stream kernel so far (the launch number in `progress`)
    char* stage_q[2];  // staging of the host-buffer entry points, two sets used alternately
    char* stage_k[2];
    char* stage_v[2];
    char* stage_out[2];
    cudaStream_t copy_stream;  // host-to-device copies of the host-buffer entry points
    cudaEvent_t ev_in[2];      // the set's inputs have landed
    cudaEvent_t ev_free[2];    // the work that used the set has finished with it
    uint64_t host_calls;
    int len;                // resident slots after the work enqueued so far
    int64_t n_full_tokens;  // full-phase tokens enqueued so far
    int64_t launches;
    int device;
    int sm_count;
    int smem_optin;  // max dynamic shared memory per block (opt-in)
    int tc_ready;    // tensor maps below are valid (bfloat16, head_dim 128)
    alignas(64) unsigned char tmap_k[128];  // CUtensorMap of the MK plane
    alignas(64) unsigned char tmap_v[128];  // CUtensorMap of the MV value plane
    alignas(64) unsigned char tmap_lo[128]; // CUtensorMap of the MV residual plane
};

namespace bct {

// One token for every unit: fill-phase append + read, or read + soft write.
// `len` is the number of resident slots before the token; do_write = 0 suppresses the
// soft write (literal first-token branch of Algorithm 1).  Returns the number of
// kernels launched (>= 1) or a negative value with *err set.
int launch_decode(const bct_cache* c, const StepIO& io, int len, int do_write, cudaStream_t stream,
                  cudaError_t* err);

// Whether launch_decode has a kernel for these parameters (shape limits of the library).
bool decode_supported(const bct_params_t& p, int smem_optin, const char** why);

// Tensor-core (tcgen05 + TMA) decode path: bfloat16, head_dim 128, group <= 15.
bool tc_prepare(bct_cache* c);          // encode the planes' tensor maps; false if unavailable
bool tc_eligible(const bct_cache* c);   // this cache's decode steps run on the tensor path
int launch_decode_tc(const bct_cache* c, const StepIO& io, int len, int do_write, cudaStream_t stream,
                     cudaError_t* err);

// Chunked tensor-core stream kernel (bfloat16, head_dim 128, G <= 7, C <= 16384):
// tokens per chunk for this cache, or 0 when the kernel does not apply.
int stream_chunk_tokens(const bct_cache* c);
// n_chunks whole chunks starting at token t_begin of the [B][T][H][d] step arrays.  fill_len < 0:
// the cache is full and every token is a read plus a soft write; fill_len >= 0: the cache holds
// fill_len slots, each chunk is appended (fill_len + n_chunks * Tc <= capacity) and read causally.
// eta: step size of each token's write, [B][T][Hkv] floats, or NULL.  write_only: the form without read
// queries and outputs (q and out unused; chunks of up to 128 tokens), full cache only.  tc_tokens: tokens per
// chunk, a multiple of 8 (16 for the write-only form) up to the cache's default, or 0 for that default; with a
// full cache the tokens of the last chunk that lie past T are zero-filled and store nothing.
int launch_stream_tc(const bct_cache* c, const void* q, const void* k, const void* v, void* out, int64_t T,
                     const float* eta, int64_t t_begin, int64_t n_chunks, int fill_len, int write_only, int tc_tokens,
                     cudaStream_t stream, cudaError_t* err);

// Backward of UpdateKV in its token-parallel form (bct_update_bwd.cu): bfloat16 caches, head_dim 128,
// 128..16384 slots.  wq, wv [B][T][Hkv][128] bfloat16, d_mv = dL/dMV_N [B][Hkv][C][128] bfloat16; outputs float:
// d_wq, d_wv [B][T][Hkv][128], d_mk [B][Hkv][C][128] (zeroed here, may be NULL), d_eta [B][T][Hkv] (may be NULL).
bool update_bwd_supported(const bct_cache* c);
int launch_update_bwd(const bct_cache* c, const void* wq, const void* wv, const float* eta, const void* d_mv, int64_t T,
                      float* d_wq, float* d_wv, float* d_mk, float* d_eta, cudaStream_t stream, cudaError_t* err);

// The projections in front of the layer (bct_project.cu): q = x W_q^T, k = x W_wq^T, v = x W_wv^T for
// n_tokens rows of x, bfloat16 throughout; status may be NULL.
cudaError_t launch_project(long long n_tokens, int d_model, int n_q, int n_kv, const void* x, const void* w_q,
                           const void* w_wq, const void* w_wv, void* q, void* k, void* v, int* status, int device,
                           int sm_count, int smem_optin, cudaStream_t stream);

// Set the calling thread's bct_last_error() message (for entry points outside bct_api.cu).
void set_last_error(const char* msg);
// BCT_OK if `c` is a handle bct_cache_create gave out and bct_cache_destroy has not taken back (looked up
// in the list of live handles, not dereferenced); otherwise the status to return, with the message set.
bct_status_t check_live_handle(const bct_cache* c);

// State import / export.
cudaError_t launch_import(const bct_cache* c, const void* k_in, const void* v_in, int v_dtype, int len,
                          cudaStream_t stream);
cudaError_t launch_export(const bct_cache* c, void* k_out, void* v_out, int v_dtype, cudaStream_t stream);
// One block whose bounded wait runs out and reports BCT_ERR_TIMEOUT (site 99) to the status words.
cudaError_t launch_wait_selftest(const bct_cache* c, cudaStream_t stream);

// Status area of the workspace (kAlign bytes of ints): word 0 = status code, word 1 = site of the
// first timeout, words 2-3 = 64-bit count of MV rows stored back by the kernels.
constexpr int kStatusRowsWord = 2;

}  // namespace bct
