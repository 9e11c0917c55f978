/*
 * bct.h: C ABI of the bounded-cache attention library for NVIDIA B200 (sm_100a).
 *
 * One attention layer of a Bounded-Cache Transformer keeps, per (sequence, kv-head)
 * "unit", a key vector sequence MK and a key-value vector sequence MV of a predefined
 * number of slots M (Method, "Model Structure"); here M is called `capacity` (C).
 * Per token, every query head of the unit reads the resident slots with softmax
 * attention, and the update rule of the paper then rewrites MV in place
 * (Method step 4, Algorithm 1, Illustration step 3):
 *
 *     read :  o_g  = softmax(read_scale  * q_g . MK^T) . MV_{t-1}       g = 0..G-1
 *     write:  MV_t = MV_{t-1} + softmax(write_scale * k_t . MK^T)^T . v_t
 *
 * q_g are the token's read queries (G = n_q_heads / n_kv_heads per unit), k_t is the
 * paper's write query wq_t and v_t its write key-value vector wv_t; the projections
 * that produce them (Algorithm 1, first two statements of the loop) are upstream of
 * this library.  MK is never assigned by Algorithm 1 and is frozen once resident.
 * While fewer than `capacity` slots are resident (a cache created with
 * init_len < capacity), a token's (k_t, v_t) is appended at slot `len`, the read covers
 * the len+1 resident slots, and no soft write happens.
 *
 * General conventions
 *  - Every pointer marked DEVICE is a device address on the current CUDA device,
 *    16-byte aligned, in memory the caller owns.  Pointers marked HOST are host
 *    addresses (pinned memory makes the copies asynchronous).
 *  - The library never allocates or frees device memory: all device storage is the
 *    caller's workspace given to bct_cache_create.
 *  - Every call validates its arguments on the host before enqueuing anything and
 *    returns a bct_status_t.  A call refused with BCT_ERR_INVALID_ARG, BCT_ERR_UNSUPPORTED
 *    or BCT_ERR_STATE has enqueued nothing and leaves the cache as it was.  BCT_ERR_CUDA
 *    means the CUDA runtime refused a launch or a copy: a call that covers several
 *    launches (bct_prefill_stream and the calls built on it split T tokens into chunk
 *    and single-token launches) may then have enqueued a prefix of its tokens; that
 *    prefix is applied in full, bct_cache_len and the token counters describe exactly
 *    the tokens enqueued, and the cache stays consistent and usable.
 *    bct_last_error() gives a thread-local message for the last failure.
 *  - Work is enqueued on the `cuda_stream` argument (a cudaStream_t passed as void*;
 *    NULL is the default stream) and the call returns without synchronising, except
 *    where stated.
 *  - A handle is not thread-safe; different handles are independent.  The library keeps a
 *    mutex-guarded list of its live handles, so that a handle passed in after
 *    bct_cache_destroy is answered with BCT_ERR_STATE without being dereferenced.
 *  - No environment variable is read.
 *  - `len` (resident slots) is the same for every sequence of the batch.
 */
#ifndef BCT_H_
#define BCT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum bct_status {
    BCT_OK = 0,
    BCT_ERR_INVALID_ARG = 1, /* NULL / misaligned pointer, out-of-range size */
    BCT_ERR_UNSUPPORTED = 2, /* a shape or flag the library has no kernel for */
    BCT_ERR_STATE = 3,       /* destroyed or corrupted handle */
    BCT_ERR_CUDA = 4,        /* a CUDA runtime call failed; see bct_last_error() */
    BCT_ERR_TIMEOUT = 5      /* a bounded device-side wait gave up (bct_cache_status) */
} bct_status_t;

typedef enum bct_dtype {
    BCT_F32 = 0, /* cache planes and step vectors in float */
    BCT_BF16 = 1 /* cache planes and step vectors in bfloat16, fp32 accumulation;
                    MV additionally carries a bfloat16 residual plane so that the
                    accumulated state keeps about 16 significand bits */
    ,
    BCT_BF16_PAIR = 2 /* checkpoint format of a bfloat16 cache's MV only (export / import):
                         one 32-bit word per element, value plane bits in the high half,
                         residual plane bits in the low half; lossless */
} bct_dtype_t;

/* flags */
#define BCT_FLAG_SKIP_FIRST_WRITE 1u /* Algorithm 1's literal "if t = 1": the first
                                        full-phase token leaves MV unchanged */
#define BCT_FLAG_WRITE_THEN_READ 2u  /* the token's read sees its own write */
#define BCT_FLAG_DENSE_WRITE 4u      /* rewrite every slot, whatever its write weight */
#define BCT_FLAG_PRECISE_READ 16u     /* bfloat16 cache: the read uses MV's value plus its
                                        residual (one more plane streamed per token; in the
                                        chunked stream kernel one more product per tile); for
                                        states whose magnitude makes a bfloat16 ulp matter */
#define BCT_FLAG_CUDA_CORES 32u       /* keep every decode step on the CUDA-core kernel (the
                                        tensor-core kernel serves bfloat16, head_dim 128,
                                        G <= 15, C >= 128 by default) */
#define BCT_FLAG_OUT_F32 8u          /* `out` is float (the fp32 accumulator, unrounded)
                                        whatever the cache dtype */

typedef struct bct_params {
    int32_t batch;      /* B  >= 1 sequences */
    int32_t n_q_heads;  /* Hq >= 1, a multiple of n_kv_heads; G = Hq / Hkv <= 8 on the CUDA-core
                           kernel, <= 15 on the tensor-core kernel */
    int32_t n_kv_heads; /* Hkv >= 1; one (MK, MV) memory per (sequence, kv-head) */
    int32_t head_dim;   /* d in {64, 128} */
    int32_t capacity;   /* C >= 1: the paper's predefined number of slots M */
    int32_t dtype;      /* bct_dtype_t */
    float read_scale;   /* <= 0 selects 1/sqrt(head_dim) */
    float write_scale;  /* <= 0 selects 1.0 (Algorithm 1 prints no scale) */
    int32_t init_len;   /* resident slots at create, 0..C; C is the paper's full-size MV_0 */
    uint32_t flags;     /* BCT_FLAG_* */
    float write_eps;    /* a slot whose write weight ww_j is below this is not rewritten
                           (its increment ww_j * v_t is dropped), in every entry point:
                           decode steps, stream chunks and bct_update_kv alike;
                           <= 0 selects 2^-24.  Ignored with BCT_FLAG_DENSE_WRITE.  With
                           BCT_FLAG_WRITE_THEN_READ the token's own read sees the slots
                           actually rewritten (the tensor-core decode kernel adds the
                           dropped slots' share as well: at most write_eps * |eta_t v_t|). */
    int32_t max_stream; /* largest T a later bct_prefill_stream_host call may pass;
                           sizes the staging area of the host-buffer entry points.
                           <= 0 selects 1. */
} bct_params_t;

typedef struct bct_cache bct_cache_t; /* opaque, host-side */

/* Library version as major*10000 + minor*100 + patch. */
int32_t bct_version(void);

/* Message of the calling thread's last failed call ("" if none).  Never NULL. */
const char *bct_last_error(void);

/*
 * Size and alignment of the device workspace a cache with these parameters needs
 * (Method, "Model Structure": MK and MV of M slots each, per unit; plus the bfloat16
 * residual plane, the status words, one progress word per (sequence, kv-head) unit and the staging
 * area of the *_host entry points).
 * The size depends on the parameters only and never grows afterwards, which is the
 * bounded-memory property of the method ("Fixed-Length Cache").
 */
bct_status_t bct_cache_bytes(const bct_params_t *params, size_t *bytes, size_t *align);

/*
 * Build a cache over caller-owned device memory and import its initial state.
 *   workspace  DEVICE, `bytes` >= bct_cache_bytes, aligned as bct_cache_bytes says;
 *              owned by the caller, must outlive the handle; the library writes to it.
 *   mk_init    DEVICE [B][Hkv][init_len][d] in `dtype`: the paper's MK (rows beyond
 *              init_len do not exist yet).  NULL allowed iff init_len == 0.
 *   mv_init    DEVICE, same shape: the paper's MV_0.  NULL with init_len > 0 means
 *              zeros (one of the two initialisations Method, "Model Structure" allows).
 * The import is enqueued on cuda_stream.  On success *out receives the handle.
 */
bct_status_t bct_cache_create(const bct_params_t *params, void *workspace, size_t bytes,
                              const void *mk_init, const void *mv_init, void *cuda_stream,
                              bct_cache_t **out);

/*
 * One token per sequence (Method steps 2-5 for the write, softmax attention for the read).
 *   q    DEVICE [B][Hq][d]   read queries; heads h*G .. h*G+G-1 belong to kv-head h
 *   k    DEVICE [B][Hkv][d]  write queries wq_t (appended as keys during the fill phase)
 *   v    DEVICE [B][Hkv][d]  write key-value vectors wv_t
 *   out  DEVICE [B][Hq][d]   attention outputs, written by the call
 * all contiguous, in the cache's dtype (out in float with BCT_FLAG_OUT_F32).  The cache advances by one token.
 */
bct_status_t bct_decode_step(bct_cache_t *cache, const void *q, const void *k, const void *v,
                             void *out, void *cuda_stream);

/*
 * T tokens per sequence, equivalent to T successive bct_decode_step calls within
 * rounding (Algorithm 1's loop over t = 1..N; with out == NULL it is UpdateKV itself,
 * which returns only the final MV_N).
 *   q    DEVICE [B][T][Hq][d]
 *   k,v  DEVICE [B][T][Hkv][d]
 *   out  DEVICE [B][T][Hq][d] or NULL
 * May be called repeatedly; successive calls concatenate.  T >= 1.  With out == NULL and a full cache
 * the call takes the write-only route of bct_update_kv (q is then not read).
 */
bct_status_t bct_prefill_stream(bct_cache_t *cache, const void *q, const void *k, const void *v,
                                void *out, int64_t T, void *cuda_stream);

/*
 * The two calls above with a step size for each token's write (Features, "Learning Rate
 * Adaptation": the step size is adjusted for each token; the paper prints no formula, so
 * the step size is an input and scales the increment of Method step 4):
 *     MV_t = MV_{t-1} + eta_t * ww_t^T . wv_t
 *   eta  DEVICE float [B][Hkv] (decode) / [B][T][Hkv] (stream), 4-byte aligned, read by
 *        the kernels of this call only; NULL means all ones, which is the call above.
 * Tokens of the fill phase are appended as they are and ignore eta; with
 * BCT_FLAG_WRITE_THEN_READ the token's own read sees the scaled write.  write_eps is
 * compared with ww_t, not with eta_t * ww_t.  Everything else as in the calls above.
 */
bct_status_t bct_decode_step_eta(bct_cache_t *cache, const void *q, const void *k, const void *v,
                                 const float *eta, void *out, void *cuda_stream);
bct_status_t bct_prefill_stream_eta(bct_cache_t *cache, const void *q, const void *k, const void *v,
                                    const float *eta, void *out, int64_t T, void *cuda_stream);

/*
 * Algorithm 1 itself, procedure UpdateKV: the write queries and write key-value vectors of T tokens
 * go into the state, MV_N = MV_0 + sum_t eta_t ww_t^T wv_t, and nothing is read.  The same state as
 * bct_prefill_stream_eta with out == NULL (within rounding), in chunks of up to 128 tokens whose
 * write weights are formed together (Key Implementation Aspects, "Optimized for Parallelism": MK is
 * never assigned, so the tokens' write weights do not depend on one another).
 *   wq   DEVICE [B][T][Hkv][d]  write queries     wv  DEVICE [B][T][Hkv][d]  write key-value vectors
 *   eta  DEVICE float [B][T][Hkv] or NULL (all ones)
 * Needs a full cache (the paper's full-size MV_0; BCT_ERR_STATE otherwise) of the shape the chunked
 * tensor-core kernel serves: bfloat16, head_dim 128, 128..16384 slots, no BCT_FLAG_SKIP_FIRST_WRITE
 * (BCT_ERR_UNSUPPORTED otherwise: use bct_prefill_stream with out == NULL).
 */
bct_status_t bct_update_kv(bct_cache_t *cache, const void *wq, const void *wv, const float *eta, int64_t T,
                           void *cuda_stream);

/*
 * Backward of bct_update_kv (Key Implementation Aspects, "Optimized for Parallelism": token-level
 * parallel training; Algorithm 1 as the forward).  For a scalar loss L and G = dL/dMV_N, with
 * ww_t = softmax(write_scale * wq_t . MK^T) of the cache's resident MK:
 *     r_t = sum_j ww_tj G_j      d_wv_t = eta_t r_t      d_eta_t = <wv_t, r_t>
 *     ds_tj = write_scale * ww_tj * (eta_t <wv_t, G_j> - eta_t d_eta_t)
 *     d_wq_t = sum_j ds_tj MK_j      d_mk_j = sum_t ds_tj wq_t      dL/dMV_0 = G (not written: it is d_mv)
 * Slots whose write weight is below write_eps are left out of r_t and of <wv_t, G_j>, as the forward
 * leaves their increments out.  The cache is read (MK only), not modified, and need not hold the MV_0
 * of the forward call: the state does not enter the gradients.
 *   wq, wv  DEVICE bfloat16 [B][T][Hkv][d]   the forward call's inputs
 *   eta     DEVICE float [B][T][Hkv] or NULL (all ones)
 *   d_mv    DEVICE bfloat16 [B][Hkv][C][d]   G
 *   d_wq, d_wv  DEVICE float [B][T][Hkv][d], written
 *   d_mk    DEVICE float [B][Hkv][C][d], written (zeroed, then summed with atomic adds: the order of the
 *           additions, hence the last bits, may differ from run to run when T > 128), or NULL
 *   d_eta   DEVICE float [B][T][Hkv], written, or NULL
 * bfloat16 operands, fp32 accumulation.  Needs a full cache of the shape the chunked kernels serve
 * (bfloat16, head_dim 128, 128..16384 slots): BCT_ERR_STATE / BCT_ERR_UNSUPPORTED otherwise.
 */
bct_status_t bct_update_kv_backward(bct_cache_t *cache, const void *wq, const void *wv, const float *eta,
                                    const void *d_mv, int64_t T, float *d_wq, float *d_wv, float *d_mk,
                                    float *d_eta, void *cuda_stream);

/*
 * The projections in front of the layer (Algorithm 1, first two statements of the loop body:
 * wq_t = W_wq x_t and wv_t = W_wv x_t; the read query q_t = W_q x_t of the attention layer
 * likewise), for a block of tokens, as one tensor-core contraction:
 *     q = x W_q^T   [n_tokens][n_q]      k = x W_wq^T, v = x W_wv^T   [n_tokens][n_kv]
 *   x      DEVICE bfloat16 [n_tokens][d_model]      one row per token (tokens of all sequences, [B][T] order)
 *   w_q    DEVICE bfloat16 [n_q][d_model]           one row per output feature, n_q = Hq * head_dim
 *   w_wq   DEVICE bfloat16 [n_kv][d_model]          n_kv = Hkv * head_dim
 *   w_wv   DEVICE bfloat16 [n_kv][d_model]
 *   q,k,v  DEVICE bfloat16, written by the call: exactly the step arrays bct_prefill_stream reads
 * fp32 accumulation, one rounding to bfloat16.  d_model a multiple of 8, n_q and n_kv multiples of 32,
 * every pointer 16-byte aligned; sm_100 devices only (BCT_ERR_UNSUPPORTED elsewhere).  Asynchronous on
 * cuda_stream; allocates nothing.
 */
bct_status_t bct_project_qkv(int64_t n_tokens, int32_t d_model, int32_t n_q, int32_t n_kv, const void *x,
                             const void *w_q, const void *w_wq, const void *w_wv, void *q, void *k, void *v,
                             void *cuda_stream);

/*
 * One layer call on the tokens themselves: the projections above, then bct_prefill_stream_eta on
 * their results (Algorithm 1's loop body from x_t to MV_t, plus the read).  bfloat16 caches only.
 *   x        DEVICE bfloat16 [B][T][d_model]
 *   eta      DEVICE float [B][T][Hkv] or NULL (all ones)
 *   scratch  DEVICE, 256-byte aligned, at least bct_layer_scratch_bytes(cache, T) bytes: holds q, k, v
 *            between the two steps; owned by the caller, free for reuse once the stream has passed the call
 *   out      DEVICE [B][T][Hq][d] or NULL
 */
bct_status_t bct_layer_scratch_bytes(const bct_cache_t *cache, int64_t T, size_t *bytes);
bct_status_t bct_layer_forward(bct_cache_t *cache, const void *x, const void *w_q, const void *w_wq,
                               const void *w_wv, int32_t d_model, const float *eta, void *scratch,
                               size_t scratch_bytes, void *out, int64_t T, void *cuda_stream);

/*
 * A stack of layers (Method, "Model Structure": the mechanism sits in every attention layer of the
 * decoder): layer 0 reads x, layer l > 0 reads the outputs of layer l - 1 taken as its tokens,
 * [B][T][Hq * d] of layer l - 1 = [B][T][d_model] of layer l; each layer is one bct_layer_forward on its own
 * cache.  No residual path, normalisation or feed-forward block is applied between the layers: those are
 * outside this library.
 *   caches   HOST array of n_layers handles (bfloat16, the same batch, without BCT_FLAG_OUT_F32)
 *   w_q, w_wq, w_wv   HOST arrays of n_layers DEVICE pointers: layer l's weights, [Hq_l * d][d_model_l] etc.,
 *            d_model_0 = d_model, d_model_l = Hq_(l-1) * head_dim
 *   scratch  DEVICE, 256-byte aligned, at least bct_stack_scratch_bytes bytes
 *   out      DEVICE [B][T][Hq][d] of the last layer
 * BCT_ERR_CUDA after the first layers have been enqueued leaves those layers' caches advanced by T tokens.
 */
bct_status_t bct_stack_scratch_bytes(bct_cache_t *const *caches, int32_t n_layers, int64_t T, size_t *bytes);
bct_status_t bct_stack_forward(bct_cache_t *const *caches, int32_t n_layers, const void *x, int32_t d_model,
                               const void *const *w_q, const void *const *w_wq, const void *const *w_wv,
                               void *scratch, size_t scratch_bytes, void *out, int64_t T, void *cuda_stream);

/*
 * Host-buffer forms of bct_decode_step and bct_prefill_stream: the same shapes, but q, k, v and out are
 * HOST pointers.  The inputs are copied into the workspace's staging area (two sets, used
 * alternately, on a copy stream the handle owns, so that one call's copies overlap the
 * previous call's kernel), the step runs on cuda_stream after them, and out is copied back
 * on cuda_stream; the call returns without synchronising, so out is valid once cuda_stream
 * has drained, and q, k, v must stay unchanged until then.  T must not exceed the
 * max_stream given at create.
 */
bct_status_t bct_decode_step_host(bct_cache_t *cache, const void *q, const void *k, const void *v,
                                  void *out, void *cuda_stream);
bct_status_t bct_prefill_stream_host(bct_cache_t *cache, const void *q, const void *k,
                                     const void *v, void *out, int64_t T, void *cuda_stream);

/*
 * bct_prefill_stream_host for callers that cannot allocate device memory.  (The paper has
 * no counterpart: this is plumbing of this library, not a step of the method.)
 *
 * bct_prefill_stream_host stages q, k, v and out in the workspace, in an area whose size the
 * caller fixed with max_stream before allocating the workspace.  Some callers can never
 * enlarge it afterwards because they cannot call cudaMalloc at all: code that runs inside a
 * memory pool frozen at start-up (a latency-bound serving loop), a plug-in that owns only
 * the arena its host application handed it, a process whose other libraries have taken the
 * rest of the device.  This call uses a staging area built into the library instead: one
 * file-scope device array of BCT_STATIC_STAGE_BYTES that every GPU holds from the moment
 * the library is loaded until the process exits.  It allocates and frees nothing.
 *
 *   q, k, v, out  HOST pointers, shapes and meaning as in bct_prefill_stream_host;
 *                 out must not be NULL.
 *   T             tokens per sequence; the rounded-up sizes of q, k, v and out for T tokens
 *                 must fit BCT_STATIC_STAGE_BYTES together, else BCT_ERR_INVALID_ARG and
 *                 nothing is enqueued (bct_last_error() gives the sizes).  max_stream does
 *                 not limit T here.
 * The cache's device must be the current device.  The first call on each device looks up
 * the array's device address (cudaGetSymbolAddress); make that first call outside any
 * stream capture.  The array is shared by every cache and every call on that device and
 * keeps the previous call's bytes; this call overwrites every byte it later reads, so
 * nothing has to be cleared, but two calls whose work overlaps on the GPU (different
 * streams without ordering, or different threads) race on it: order them on one stream.
 * Results are those of bct_prefill_stream_host.
 */
#define BCT_STATIC_STAGE_BYTES (8u << 20)
bct_status_t bct_prefill_stream_host_static(bct_cache_t *cache, const void *q, const void *k,
                                            const void *v, void *out, int64_t T,
                                            void *cuda_stream);

/* Resident slots (0..C) after the work enqueued so far. Host bookkeeping; no sync. */
bct_status_t bct_cache_len(const bct_cache_t *cache, int32_t *len);

/*
 * Copy the state out in the canonical layout (Method step 5, the store of the updated
 * sequence, made visible): k_out DEVICE [B][Hkv][C][d] in the cache dtype, v_out DEVICE
 * [B][Hkv][C][d] in v_dtype (BCT_F32 gives the bfloat16 value plus its residual,
 * exactly; BCT_BF16 the rounded value; BCT_BF16_PAIR both planes bit for bit).  Rows
 * >= len are written as zeros.  Either pointer may be NULL to skip that plane.
 */
bct_status_t bct_cache_export(bct_cache_t *cache, void *k_out, void *v_out, int32_t v_dtype,
                              void *cuda_stream);

/*
 * Replace the state: k_in DEVICE [B][Hkv][len][d] in the cache dtype, v_in DEVICE
 * [B][Hkv][len][d] in v_dtype (NULL = zeros), 0 <= len <= C.  Counters of tokens seen
 * are kept.  export followed by import into a fresh cache resumes bit-exactly with
 * v_dtype BCT_BF16_PAIR (bfloat16 cache) or BCT_F32 (float cache); a bfloat16 cache
 * re-imported from BCT_F32 holds the same values but may split a few of them
 * differently between the value and residual planes.
 */
bct_status_t bct_cache_import(bct_cache_t *cache, const void *k_in, const void *v_in,
                              int32_t v_dtype, int32_t len, void *cuda_stream);

/*
 * Synchronise cuda_stream and report the device-side status word: BCT_OK, or
 * BCT_ERR_TIMEOUT if a bounded wait inside a kernel gave up (the affected step's
 * results are then undefined; the context stays usable).  The only call that blocks.
 */
bct_status_t bct_cache_status(bct_cache_t *cache, void *cuda_stream);

/* Set the device-side status word back to BCT_OK (enqueued on cuda_stream, no synchronisation):
 * after a reported BCT_ERR_TIMEOUT the cache can be re-imported and used again. */
bct_status_t bct_cache_status_clear(bct_cache_t *cache, void *cuda_stream);

/*
 * Rows of MV that the kernels of this cache have stored back so far (Method step 5: the store of the
 * updated sequence): decode steps count the slots whose write weight reached write_eps (every slot
 * with BCT_FLAG_DENSE_WRITE), the chunked stream kernel rebuilds whole tiles and counts every slot
 * of every chunk; appended fill-phase slots are not counted.  Synchronises cuda_stream like
 * bct_cache_status.  The fraction w = rows / (units * full-phase tokens * capacity) is the share of
 * MV the update rule rewrites per token, the term w*C*d*s of the bytes a decode step must move.
 *   rows  HOST, receives the count (64 bits).
 */
bct_status_t bct_cache_rows_rewritten(bct_cache_t *cache, void *cuda_stream, uint64_t *rows);

/*
 * Self-test of the bounded device-side waits (no step of the method): launches one thread block on
 * cuda_stream that waits, with a limit of about a thousand polls, on a barrier in its shared memory
 * that nothing ever arrives on; the wait gives up, the block records BCT_ERR_TIMEOUT with site code
 * 99 in the cache's status word and returns normally.  Nothing faults, hangs or traps, and the cache's
 * planes are not touched.  bct_cache_status then reports BCT_ERR_TIMEOUT until
 * bct_cache_status_clear.  Asynchronous.
 */
bct_status_t bct_selftest_timeout(bct_cache_t *cache, void *cuda_stream);

/* *yes = 1 if this cache's decode steps run on the tensor-core kernel (tcgen05 + TMA tensor
 * copies: bfloat16, head_dim 128, G <= 15, 128 <= C <= 65536, no PRECISE_READ / CUDA_CORES
 * flag), 0 if on the CUDA-core kernel.  Both compute the same step (Algorithm 1 + read). */
bct_status_t bct_cache_tensor_path(const bct_cache_t *cache, int32_t *yes);

/* Number of kernels this handle has launched so far (host counter). */
bct_status_t bct_cache_launches(const bct_cache_t *cache, int64_t *launches);

/* Free the host-side handle (NULL is accepted).  Never touches the workspace, never
 * synchronises: the caller drains the stream before reusing the workspace. */
bct_status_t bct_cache_destroy(bct_cache_t *cache);

#ifdef __cplusplus
}
#endif
#endif /* BCT_H_ */
