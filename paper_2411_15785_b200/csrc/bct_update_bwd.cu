// Backward of Algorithm 1's procedure UpdateKV in its token-parallel form, on the sm_100a tensor path.
//
// Forward (Key Implementation Aspects, "Optimized for Parallelism": MK is never assigned, so the write
// weights of all tokens are independent and the final state is one sum over the tokens):
//     WW = softmax rows of (write_scale * Wq MK^T)          [T x C]
//     MV_N = MV_0 + WW^T diag(eta) Wv                        [C x d]
// Given G = dL/dMV_N, per (sequence, kv-head) unit and per block of 128 tokens (one CTA each):
//     R    = WW G                 [T x d]   dWv = diag(eta) R,  deta_t = <wv_t, R_t>,  delta_t = eta_t deta_t
//     A    = Wv G^T               [T x C]   what each slot's gradient row sees of each write value
//     dS   = write_scale * WW o (diag(eta) A - delta)        (softmax Jacobian, row by row)
//     dWq  = dS MK                [T x d]
//     dMK += dS^T Wq              [C x d]   summed over the token blocks of the unit (fp32 atomics)
// and dL/dMV_0 = G.  With a write threshold the slots with ww < write_eps are dropped from R and A
// (the forward drops their increments; the mask is piecewise constant).
// Five contractions per (token block, 128-slot tile), all tcgen05.mma with M = 128 and fp32 accumulators
// in tensor memory; the softmax statistics need the whole row, so the tiles are walked three times:
//   pass 1  S = Wq MK_t^T                      -> row maxima and sums
//   pass 2  S again -> WW_t (bfloat16), R += WW_t G_t
//   pass 3  S and A_t = Wv G_t^T -> dS_t (bfloat16), dWq += dS_t MK_t, dMK_t = dS_t^T Wq -> atomics
//   warps 0-15  four threads per token row (= tensor-memory lane), 32 accumulator columns each: statistics, the
//               WW / dS operand, outputs
//   warp 16     one thread issues the TMA loads (four tile buffers, loaded one tile ahead) and every MMA
// Software pipeline: the row threads hold the operand of tile t in registers while the products of tile t-1 read
// the operand buffer, and the scores of the tile after are issued before the products of the current one, so
// that exponentials and tensor work overlap.  The roles meet at block-wide barriers plus one mbarrier (scores
// consumed); the issuing thread's waits on the TMA and MMA barriers are bounded, a timeout sets the status word
// and the kernel runs to its end.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "bct_internal.h"
#include "bct_tc.cuh"

namespace bct {
namespace {

constexpr int kBwRows = 128;                 // tokens per block = operand rows = tensor-memory lanes
constexpr int kBwRowThreads = 4 * kBwRows;   // four threads per row
constexpr int kBwThreads = kBwRowThreads + 32;  // + the issuing warp
constexpr int kBwTile = 128;                 // slots per tile
constexpr int kBwHalf = 128 * 128;           // 64 columns (128 bytes) x 128 rows
constexpr int kBwTileBytes = 2 * kBwHalf;
constexpr int kBwRing = 4;                   // tile buffers
constexpr float kBwNegBig = -3.0e38f;
// tensor-memory columns
constexpr int kColS = 0;      // scores [token] x [slot]; buffer 0 of the scores in passes 1 and 2
constexpr int kColA = 128;    // A = Wv G_t^T [token] x [slot] in pass 3; buffer 1 of the scores in passes 1 and 2
constexpr int kColR = 256;    // R (pass 2), then dWq (pass 3)   [token] x [d]
constexpr int kColM = 384;    // dMK of one tile   [slot] x [d]

struct BwArgs {
    float* d_wq;
    float* d_wv;
    float* d_mk;
    float* d_eta;
    const float* eta;
    const char* wv;   // the write key-value vectors themselves, for deta_t = <wv_t, R_t>
    int* status;
    int C, Hkv, T, n_blocks;
    float write_scale, write_eps;
};

struct BwSmem {
    int wq, wv, op, ring, bars, misc, total;
};
__host__ __device__ inline BwSmem bw_smem() {
    BwSmem L;
    int off = 0;
    L.wq = off;       // [2 halves][128 tokens][128 B]: the block's write queries
    off += kBwTileBytes;
    L.wv = off;       // ... and write key-value vectors
    off += kBwTileBytes;
    L.op = off;       // WW_t (pass 2) / dS_t (pass 3) of one tile, bfloat16, rows = tokens; between the passes: row statistics
    off += kBwTileBytes;
    L.ring = off;     // MK and G tiles
    off += kBwRing * kBwTileBytes;
    L.bars = off;
    off += 8 * 8;
    L.misc = off;
    off += 64;
    L.total = off + 1024;  // slack to align the base to 1024 bytes
    return L;
}

__device__ __forceinline__ float bw_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__global__ void __launch_bounds__(kBwThreads, 1)
update_bwd_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmG,
                  const __grid_constant__ CUtensorMap tmWq, const __grid_constant__ CUtensorMap tmWv, const BwArgs a) {
    extern __shared__ unsigned char bw_smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(bw_smem_raw) + 1023) & ~uintptr_t(1023));
    const BwSmem L = bw_smem();
    unsigned char* wqb = smem + L.wq;
    unsigned char* wvb = smem + L.wv;
    unsigned char* opb = smem + L.op;
    unsigned char* ring = smem + L.ring;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L.bars);   // [4] tile landed; [4]: the block's operands landed
    uint64_t* mma_done = full + 5;                                   // every MMA issued so far is complete
    uint64_t* sa_free = full + 6;                                    // pass 3: the scores and A of a tile are in registers (512 arrivals)
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L.misc);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L.misc + 8);
    float* xch = reinterpret_cast<float*>(opb);                      // [4 quarters][128 rows][2]: exchange between the four threads of a row

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int u = blockIdx.x / a.n_blocks;
    const int blk = blockIdx.x - u * a.n_blocks;
    const int b = u / a.Hkv, h = u - b * a.Hkv;
    const int t0 = blk * kBwRows;
    const int nt = (a.C + kBwTile - 1) / kBwTile;
    const bool issuer = (tid == kBwRowThreads);
    constexpr int kIssuerWarp = kBwRowThreads / 32;

    if (tid == 0) {
        for (int i = 0; i < 5; ++i) mbar_init(&full[i], 1);
        mbar_init(mma_done, 1);
        mbar_init(sa_free, kBwRowThreads);
        *abort_flag = 0;
        fence_mbar_init_cluster();
    }
    if (warp == kIssuerWarp) tmem_alloc(tmem_slot, 512);
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

#define BW_WAIT(bar, parity, site)                                 \
    if (!mbar_wait_abortable(bar, (parity) & 1, abort_flag)) {     \
        report_timeout(a.status, site);                            \
        *abort_flag = 1;                                           \
    }

    // ---- the issuing thread's tools: tile buffers with a use count each (the phase of their barriers) ----
    uint32_t use[kBwRing] = {0, 0, 0, 0};  // loads issued into each buffer
    uint32_t n_mma = 0, n_sa = 0;          // commits waited for, score hand-overs waited for
    auto buf_ptr = [&](int bf) { return ring + (size_t)bf * kBwTileBytes; };
    auto load_tile = [&](int bf, bool is_g, int t) {   // tile t of MK (or of G) into buffer bf
        mbar_arrive_expect_tx(&full[bf], kBwTileBytes);
        tma_load_3d(buf_ptr(bf), is_g ? &tmG : &tmK, 0, t * kBwTile, u, &full[bf]);
        tma_load_3d(buf_ptr(bf) + kBwHalf, is_g ? &tmG : &tmK, 64, t * kBwTile, u, &full[bf]);
        ++use[bf];
    };
    auto wait_tile = [&](int bf) { BW_WAIT(&full[bf], use[bf] - 1, 81); };  // the buffer's latest load has landed
    auto commit_and_wait = [&]() {
        umma_commit(mma_done);
        BW_WAIT(mma_done, n_mma, 82);
        ++n_mma;
        tc_fence_after();
    };
    constexpr uint32_t id_kk = instr_desc_mn(128, 128, false, false);  // A (K-major) x B (K-major): scores, A
    constexpr uint32_t id_kn = instr_desc_mn(128, 128, false, true);   // A (K-major) x B (MN-major): R, dWq
    constexpr uint32_t id_nn = instr_desc_mn(128, 128, true, true);    // A (MN-major) x B (MN-major): dMK
    const DescKind dk(smem_desc(0, 16, 1024)), dmn(smem_desc(0, kBwHalf, 1024));
    // D[token][n] (+)= X[token][k] * Y[n][k], both operands K-major, k = 0..127 in eight steps
    auto mma_kk = [&](int col, const unsigned char* x, const unsigned char* y, bool accum) {
        const uint32_t xa = desc_addr16(smem_u32(x)), ya = desc_addr16(smem_u32(y));
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            const uint32_t o = ((kk >> 2) * kBwHalf + (kk & 3) * 32) / 16;
            umma_bf16(tmem_base + col, dk.at(xa + o), dk.at(ya + o), id_kk, accum || kk > 0);
        }
    };
    // D[token][n] (+)= X[token][k] * Y[k][n]: X K-major, Y stored as rows k (MN-major operand)
    auto mma_kn = [&](int col, const unsigned char* x, const unsigned char* y, bool accum) {
        const uint32_t xa = desc_addr16(smem_u32(x)), ya = desc_addr16(smem_u32(y));
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            const uint32_t o = ((kk >> 2) * kBwHalf + (kk & 3) * 32) / 16;
            umma_bf16(tmem_base + col, dk.at(xa + o), dmn.at(ya + kk * 128), id_kn, accum || kk > 0);
        }
    };
    // D[m][n] = sum_k X[k][m] * Y[k][n]: both stored as rows k (MN-major operands)
    auto mma_nn = [&](int col, const unsigned char* x, const unsigned char* y) {
        const uint32_t xa = desc_addr16(smem_u32(x)), ya = desc_addr16(smem_u32(y));
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) umma_bf16(tmem_base + col, dmn.at(xa + kk * 128), dmn.at(ya + kk * 128), id_nn, kk > 0);
    };

    if (issuer) {
        mbar_arrive_expect_tx(&full[4], 2 * kBwTileBytes);
        tma_load_4d(wqb, &tmWq, 0, h, t0, b, &full[4]);
        tma_load_4d(wqb + kBwHalf, &tmWq, 64, h, t0, b, &full[4]);
        tma_load_4d(wvb, &tmWv, 0, h, t0, b, &full[4]);
        tma_load_4d(wvb + kBwHalf, &tmWv, 64, h, t0, b, &full[4]);
        for (int t = 0; t < nt && t < kBwRing; ++t) load_tile(t, false, t);  // pass 1: MK_t in buffer t mod 4
        BW_WAIT(&full[4], 0, 80);
    }

    // ---- row threads: thread (r, cq) holds columns [32 cq, 32 cq + 32) of row r of every 128-column accumulator ----
    const int r = tid & 127;
    const int cq = (tid >> 7) & 3;
    const bool is_row = tid < kBwRowThreads;
    const bool row_valid = is_row && (t0 + r < a.T);
    const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + cq * 32;
    const float c2 = a.write_scale * 1.4426950408889634f;  // exponentials are taken in base 2
    const size_t tok = ((size_t)b * a.T + (size_t)(t0 + r)) * a.Hkv + h;  // this token's row in [B][T][Hkv]
    const float eta = (row_valid && a.eta != nullptr) ? a.eta[tok] : 1.f;
    const int sw = r & 7;  // swizzle phase of this row in the operand buffer
    // this thread's 32 slots of its row, as bfloat16, into the operand buffer (K-major, 128-byte swizzle)
    auto store_op = [&](const float* x) {
        unsigned char* row = opb + (cq >> 1) * kBwHalf + r * 128;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            *reinterpret_cast<uint4*>(row + ((((cq & 1) * 4 + j) ^ sw) * 16)) = Chunk<__nv_bfloat16>::pack(x + 8 * j);
    };

    // ---------------- pass 1: maximum and sum of every row's scaled scores (this thread: its 32 columns of every tile) ----
    // The scores of tile t + 1 are issued while the row threads work on tile t (two score buffers).
    float m = kBwNegBig, l = 0.f;
    if (issuer && nt > 0) {
        wait_tile(0);
        tc_fence_after();
        mma_kk(kColS, wqb, buf_ptr(0), false);
        commit_and_wait();
        if (4 < nt) load_tile(0, false, 4);
    }
    for (int t = 0; t < nt; ++t) {
        __syncthreads();  // the scores of tile t are complete, and tile t - 1's have been read
        if (issuer && t + 1 < nt) {
            const int bf = (t + 1) % kBwRing;
            wait_tile(bf);
            tc_fence_after();
            mma_kk(((t + 1) & 1) ? kColA : kColS, wqb, buf_ptr(bf), false);
            commit_and_wait();
            if (t + 5 < nt) load_tile(bf, false, t + 5);
        }
        if (is_row) {
            tc_fence_after();
            const int n_valid = min(kBwTile, a.C - t * kBwTile) - cq * 32;
            float x[32];
            tmem_ld32(lane_base + ((t & 1) ? kColA : kColS), x);
            float mt = kBwNegBig;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                x[i] = (i < n_valid) ? x[i] * c2 : kBwNegBig;
                mt = fmaxf(mt, x[i]);
            }
            const float mn = fmaxf(m, mt);
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                s0 += (i < n_valid) ? bw_ex2(x[i] - mn) : 0.f;
                s1 += (i + 1 < n_valid) ? bw_ex2(x[i + 1] - mn) : 0.f;
            }
            l = l * bw_ex2(m - mn) + (s0 + s1);
            m = mn;
            tc_fence_before();
        }
    }
    __syncthreads();
    // combine the four quarters of every row (through the operand buffer, idle here)
    if (is_row) {
        xch[(cq * 128 + r) * 2] = m;
        xch[(cq * 128 + r) * 2 + 1] = l;
    }
    __syncthreads();
    if (is_row) {
        float mn = m;
#pragma unroll
        for (int o = 1; o < 4; ++o) mn = fmaxf(mn, xch[(((cq + o) & 3) * 128 + r) * 2]);
        l *= bw_ex2(m - mn);
#pragma unroll
        for (int o = 1; o < 4; ++o) {
            const int idx = (((cq + o) & 3) * 128 + r) * 2;
            l += xch[idx + 1] * bw_ex2(xch[idx] - mn);
        }
        m = mn;
    }
    const float inv_l = 1.f / l;

    // ---------------- pass 2: WW_t as an operand, R += WW_t G_t ----------------
    // MK_t sits in buffer t & 1, G_t in buffer 2 + (t & 1).  Iteration t stores the weights of tile t (held in
    // registers since the iteration before) and, while R += WW_t G_t and the scores of tile t + 2 run, takes the
    // weights of tile t + 1 from its scores.
    float p[32];
    auto weights_of = [&](int t) {   // normalised, thresholded write weights of tile t, this thread's 32 slots
        const int n_valid = min(kBwTile, a.C - t * kBwTile) - cq * 32;
        tmem_ld32(lane_base + ((t & 1) ? kColA : kColS), p);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const float ww = (i < n_valid) ? bw_ex2(fmaf(p[i], c2, -m)) * inv_l : 0.f;
            p[i] = ww >= a.write_eps ? ww : 0.f;   // a dropped slot's increment does not depend on anything
        }
    };
    __syncthreads();  // the statistics have been read out of the operand buffer
    if (issuer && nt > 0) {
        load_tile(0, false, 0);
        load_tile(2, true, 0);
        if (nt > 1) {
            load_tile(1, false, 1);
            load_tile(3, true, 1);
        }
        wait_tile(0);
        tc_fence_after();
        mma_kk(kColS, wqb, buf_ptr(0), false);
        commit_and_wait();
        if (nt > 2) load_tile(0, false, 2);
        if (nt > 1) {
            wait_tile(1);
            tc_fence_after();
            mma_kk(kColA, wqb, buf_ptr(1), false);
        }
    }
    __syncthreads();
    if (is_row && nt > 0) {
        tc_fence_after();
        weights_of(0);
        tc_fence_before();
    }
    for (int t = 0; t < nt; ++t) {
        if (issuer) {
            commit_and_wait();  // R of tile t - 1 and the scores of tile t + 1 are complete
            if (t + 3 < nt) load_tile((t + 1) & 1, false, t + 3);
            if (t >= 1 && t + 1 < nt) load_tile(2 + ((t + 1) & 1), true, t + 1);
        }
        __syncthreads();  // the operand buffer is free
        if (is_row) {
            store_op(p);
            fence_proxy_async_smem();
        }
        __syncthreads();  // WW_t is in the operand buffer
        if (issuer) {
            wait_tile(2 + (t & 1));
            tc_fence_after();
            mma_kn(kColR, opb, buf_ptr(2 + (t & 1)), t > 0);
            if (t + 2 < nt) {
                wait_tile(t & 1);
                mma_kk((t & 1) ? kColA : kColS, wqb, buf_ptr(t & 1), false);
            }
        }
        if (is_row && t + 1 < nt) {
            tc_fence_after();
            weights_of(t + 1);
            tc_fence_before();
        }
    }
    if (issuer) commit_and_wait();
    __syncthreads();
    // R_t is complete: dwv_t = eta_t R_t, deta_t = <wv_t, R_t>, delta_t = eta_t deta_t
    float delta = 0.f;
    {
        float de = 0.f;
        if (is_row) {
            tc_fence_after();
            float x[32];
            tmem_ld32(lane_base + kColR, x);
            if (row_valid) {
                const __nv_bfloat16* vrow = reinterpret_cast<const __nv_bfloat16*>(a.wv) + tok * 128 + cq * 32;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float v8[8];
                    Chunk<__nv_bfloat16>::unpack(*reinterpret_cast<const uint4*>(vrow + j * 8), v8);
#pragma unroll
                    for (int i = 0; i < 8; ++i) de = fmaf(v8[i], x[8 * j + i], de);
                }
                float4* dst = reinterpret_cast<float4*>(a.d_wv + tok * 128 + cq * 32);
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    dst[j] = make_float4(eta * x[4 * j], eta * x[4 * j + 1], eta * x[4 * j + 2], eta * x[4 * j + 3]);
            }
            tc_fence_before();
            xch[cq * 128 + r] = de;
        }
        __syncthreads();
        if (is_row) {
            de = (xch[r] + xch[128 + r]) + (xch[256 + r] + xch[384 + r]);
            if (row_valid && cq == 0 && a.d_eta != nullptr) a.d_eta[tok] = de;
            delta = eta * de;
        }
        __syncthreads();  // the sums have been read out of the operand buffer
    }

    // ---------------- pass 3: dS_t as an operand, dWq += dS_t MK_t, dMK_t = dS_t^T Wq ----------------
    // MK_t sits in buffer t mod 3 (it is read twice: by the scores and, a tile later, by the dWq product), G_t in
    // buffer 3.  Iteration t stores dS_t (held in registers) and flushes dMK of tile t - 1; dS of tile t + 1 is taken
    // from its scores while the products of tile t run.
    auto ds_of = [&](int t) {   // dS of tile t, this thread's 32 slots, into p
        const int n_valid = min(kBwTile, a.C - t * kBwTile) - cq * 32;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            float x[16], g[16];
            tmem_ld16(lane_base + kColS + hh * 16, x);
            tmem_ld16(lane_base + kColA + hh * 16, g);
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float ww = (hh * 16 + i < n_valid) ? bw_ex2(fmaf(x[i], c2, -m)) * inv_l : 0.f;
                const float dww = ww >= a.write_eps ? eta * g[i] : 0.f;
                // the weight as pass 2 rounded it: delta was formed with those, and dww - delta cancels to
                // the last bits for the slot that holds most of the weight
                const float wr = __bfloat162float(__float2bfloat16_rn(ww));
                p[hh * 16 + i] = row_valid ? a.write_scale * wr * (dww - delta) : 0.f;   // rows past the last token add nothing
            }
        }
    };
    // the slot rows of dMK_t leave tensor memory one tile late (lanes are slots there), as atomic adds: the token
    // blocks of a unit run on different SMs
    auto flush_dmk = [&](int t) {
        const int slot = t * kBwTile + r;
        float x[32];
        tmem_ld32(lane_base + kColM, x);
        if (slot < a.C && a.d_mk != nullptr) {
            float4* dst = reinterpret_cast<float4*>(a.d_mk + ((size_t)u * a.C + slot) * 128 + cq * 32);
#pragma unroll
            for (int j = 0; j < 8; ++j) atomicAdd(dst + j, make_float4(x[4 * j], x[4 * j + 1], x[4 * j + 2], x[4 * j + 3]));
        }
    };
    if (issuer && nt > 0) {
        load_tile(0, false, 0);
        load_tile(3, true, 0);
        if (nt > 1) load_tile(1, false, 1);
        wait_tile(0);
        wait_tile(3);
        tc_fence_after();
        mma_kk(kColS, wqb, buf_ptr(0), false);
        mma_kk(kColA, wvb, buf_ptr(3), false);
        commit_and_wait();
        if (nt > 1) load_tile(3, true, 1);
    }
    __syncthreads();
    if (is_row && nt > 0) {
        tc_fence_after();
        ds_of(0);
        tc_fence_before();
        mbar_arrive(sa_free);
    }
    for (int t = 0; t < nt; ++t) {
        if (issuer) {
            BW_WAIT(sa_free, n_sa, 83);  // the scores and A of tile t are in registers
            ++n_sa;
            tc_fence_after();
            if (t + 1 < nt) {
                const int bf = (t + 1) % 3;
                wait_tile(bf);
                wait_tile(3);
                tc_fence_after();
                mma_kk(kColS, wqb, buf_ptr(bf), false);
                mma_kk(kColA, wvb, buf_ptr(3), false);
            }
            commit_and_wait();  // the products of tile t - 1 and the scores and A of tile t + 1 are complete
            if (t + 2 < nt) {
                load_tile((t + 2) % 3, false, t + 2);
                load_tile(3, true, t + 2);
            }
        }
        __syncthreads();  // the operand buffer is free, dMK of tile t - 1 is complete
        if (is_row) {
            tc_fence_after();
            if (t > 0) flush_dmk(t - 1);
            store_op(p);
            fence_proxy_async_smem();
            tc_fence_before();
        }
        __syncthreads();  // dS_t is in the operand buffer, dMK of tile t - 1 has left tensor memory
        if (issuer) {
            tc_fence_after();
            mma_kn(kColR, opb, buf_ptr(t % 3), t > 0);
            mma_nn(kColM, opb, wqb);
        }
        if (is_row && t + 1 < nt) {
            tc_fence_after();
            ds_of(t + 1);
            tc_fence_before();
            mbar_arrive(sa_free);
        }
    }
    if (issuer) commit_and_wait();
    __syncthreads();
    if (is_row) {
        tc_fence_after();
        if (nt > 0) flush_dmk(nt - 1);
        const bool store = row_valid && !*abort_flag;
        float x[32];
        tmem_ld32(lane_base + kColR, x);  // (the whole warp takes part in the load, whatever it stores)
        if (store) {
            float4* dst = reinterpret_cast<float4*>(a.d_wq + tok * 128 + cq * 32);
#pragma unroll
            for (int j = 0; j < 8; ++j) dst[j] = make_float4(x[4 * j], x[4 * j + 1], x[4 * j + 2], x[4 * j + 3]);
        }
        tc_fence_before();
    }
#undef BW_WAIT
    __syncthreads();
    if (warp == kIssuerWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// [U][C][128] bfloat16 as a 3-D tensor (d, slot, unit), boxes of 64 columns x 128 slots, 128-byte swizzle;
// rows past C read as zeros.
bool bw_plane_map(CUtensorMap* map, const void* base, int U, int C) {
    TensorMapEncodeFn fn = tensor_map_encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[3] = {128, (cuuint64_t)C, (cuuint64_t)U};
    const cuuint64_t strides[2] = {256, (cuuint64_t)C * 256};
    const cuuint32_t box[3] = {64, (cuuint32_t)kBwTile, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Step vectors [B][T][H][128] bfloat16 as (d, head, token, sequence); one box is 64 columns of one head for
// 128 tokens, landing as rows = tokens; tokens past T read as zeros.
bool bw_step_map(CUtensorMap* map, const void* base, int B, int T, int H) {
    TensorMapEncodeFn fn = tensor_map_encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[4] = {128, (cuuint64_t)H, (cuuint64_t)T, (cuuint64_t)B};
    const cuuint64_t strides[3] = {256, (cuuint64_t)H * 256, (cuuint64_t)T * H * 256};
    const cuuint32_t box[4] = {64, 1, (cuuint32_t)kBwRows, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool update_bwd_supported(const bct_cache* c) {
    const bct_params_t& p = c->p;
    return p.dtype == BCT_BF16 && p.head_dim == 128 && c->tc_ready && p.capacity >= kBwTile && p.capacity <= 16384 &&
           bw_smem().total <= c->smem_optin;
}

int launch_update_bwd(const bct_cache* c, const void* wq, const void* wv, const float* eta, const void* d_mv, int64_t T,
                      float* d_wq, float* d_wv, float* d_mk, float* d_eta, cudaStream_t stream, cudaError_t* err) {
    const bct_params_t& p = c->p;
    if (!update_bwd_supported(c) || T < 1 || T > kMaxCallTokens) {
        *err = cudaErrorInvalidConfiguration;
        return -1;
    }
    alignas(64) CUtensorMap mg, mq, mv;
    if (!bw_plane_map(&mg, d_mv, c->U, p.capacity) || !bw_step_map(&mq, wq, p.batch, (int)T, p.n_kv_heads) ||
        !bw_step_map(&mv, wv, p.batch, (int)T, p.n_kv_heads)) {
        *err = cudaErrorInvalidValue;
        return -1;
    }
    const int n_blocks = (int)((T + kBwRows - 1) / kBwRows);
    if ((long long)c->U * n_blocks > 0x7fffffffLL) {
        *err = cudaErrorInvalidConfiguration;
        return -1;
    }
    BwArgs a;
    a.d_wq = d_wq;
    a.d_wv = d_wv;
    a.d_mk = d_mk;
    a.d_eta = d_eta;
    a.eta = eta;
    a.wv = static_cast<const char*>(wv);
    a.status = c->status;
    a.C = p.capacity;
    a.Hkv = p.n_kv_heads;
    a.T = (int)T;
    a.n_blocks = n_blocks;
    a.write_scale = p.write_scale;
    a.write_eps = (p.flags & BCT_FLAG_DENSE_WRITE) ? 0.f : p.write_eps;
    int launches = 0;
    if (d_mk != nullptr) {  // the token blocks of a unit add their shares into it
        *err = cudaMemsetAsync(d_mk, 0, (size_t)c->U * p.capacity * 128 * sizeof(float), stream);
        if (*err != cudaSuccess) return -1;
    }
    const int smem = bw_smem().total;
    *err = cudaFuncSetAttribute(reinterpret_cast<const void*>(update_bwd_kernel), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                smem);
    if (*err != cudaSuccess) return -1;
    update_bwd_kernel<<<(unsigned)(c->U * n_blocks), kBwThreads, smem, stream>>>(
        *reinterpret_cast<const CUtensorMap*>(c->tmap_k), mg, mq, mv, a);
    *err = cudaGetLastError();
    if (*err != cudaSuccess) return -1;
    ++launches;
    return launches;
}

}  // namespace bct
