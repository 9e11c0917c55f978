// Decode step of the bounded-cache attention layer on the sm_100a tensor path
// (bfloat16 cache, head_dim 128, up to 7 query heads per kv-head).
//
// The two contractions of a token are small-N GEMMs against the resident tiles:
//   scores   S[slot, h]  = sum_d MK[slot, d] * Q[h, d]      h = G read queries + the write query
//                                                           (score_t = wq_t . MK^T, Algorithm 1)
//   outputs  O[d, g]     = sum_slot MV[slot, d] * P[g, slot] (softmax numerators P; read path)
// Both run as tcgen05.mma (M = 128, N = 16, K = 16) straight out of the shared-memory tiles that
// TMA tensor copies deliver (128-byte swizzle), with the accumulators in tensor memory, so the
// SM's issue slots carry only the softmax and the update rule
//   MV_t = MV_{t-1} + ww_t^T . wv_t   (Method step 4)
// on the few rows whose weight reaches write_eps.
//
// One persistent CTA per SM (or a cluster of S CTAs per unit when C > 2048 slots), three roles:
//   warp 4  producer : TMA loads of K tiles then V tiles into a ring, running ahead across units
//   warp 5  MMA      : issues the tensor-core work as tiles land; its commits free the ring stages
//   warps 0-3        : softmax statistics from tensor memory, P operand, epilogue, and the update
//                      rule from staged copies of the rows to rewrite (applied once the unit's V
//                      tiles have all been read, so the read sees MV_{t-1})
// Every wait is bounded; a timeout sets the status word and the kernel runs to its end.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <mutex>

#include "bct_internal.h"
#include "bct_tc.cuh"

namespace bct {
namespace {

constexpr int kTcThreads = 192;
constexpr int kSThreads = 128;
constexpr int kTileRows = 128;
constexpr int kHalfBytes = 128 * 128;          // 64 columns (128 bytes) x 128 rows
constexpr int kTcTileBytes = 2 * kHalfBytes;   // one 128 x 128 bfloat16 tile
constexpr int kMaxTiles = 16;                  // tiles per sub-slice: score tiles resident in tensor memory
constexpr int kMaxSliceRows = 8192;            // slots per CTA: up to 4 sub-slices of 2048, streamed one after the other
// Operand rows of the small operands (queries, softmax numerators): the N = 16 instruction shape reads 16
// rows; with up to 7 read heads 8 rows are kept and the upper 8 are whatever follows (their score / output
// columns are never read), with 8 to 15 read heads all 16 are kept.
__host__ __device__ constexpr int tc_rows(int G) { return G + 1 <= 8 ? 8 : 16; }
__host__ __device__ constexpr int tc_ptile_bytes(int G) { return 2 * tc_rows(G) * 128; }  // P operand of one tile: 2 halves
__host__ __device__ constexpr int tc_qbuf_bytes(int G) {  // Q operand: 2 halves (+ 1 KiB of zeros behind 8-row halves)
    return 2 * tc_rows(G) * 128 + (tc_rows(G) == 8 ? 1024 : 0);
}
constexpr int kScoreCols = 16;                 // tensor-memory columns per score tile (N = 16)
constexpr int kSmallTiles = 8;                 // tiles per unit in the two-CTAs-per-SM form (units of up to 1024 slots)
// The output accumulator sits behind the score tiles; a CTA takes all 512 tensor-memory columns, or 256 in the
// two-CTAs-per-SM form (an SM has 512: two resident CTAs must share them).
__host__ __device__ constexpr int tc_ocol(bool small) { return (small ? kSmallTiles : kMaxTiles) * kScoreCols; }
__host__ __device__ constexpr int tc_tmem_cols(bool small) { return small ? 256 : 512; }
constexpr int kMaxClusterTc = 8;
constexpr int kLwwCap = 512;                   // rewritten rows whose weights are kept for the deferred update
constexpr float kNegBigTc = -3.0e38f;

struct TcArgs {
    char* vhi;
    char* vlo;
    char* kplane;
    const char* q;
    const char* k;
    const char* v;
    char* out;
    int* status;
    long long q_bs;
    long long kv_bs;
    const float* eta;   // step size of each unit's write, [sequence][kv-head], or NULL (all ones)
    long long eta_bs;
    int C, len, slice_rows, S, Hkv, U, stages, lo_cap;  // lo_cap: rewritten rows staged per round
    int do_write, wtr, dense, out_f32;
    float read_scale, write_scale, write_eps;
};

struct TcSmem {
    int ring, pbuf, qbuf, wsm, list, lww, lostage, red, stat, vtb, wstat, merge, bars, total;
};
__host__ __device__ inline TcSmem tc_smem(int stages, int G, int S, int slice_rows, int lo_cap) {
    const int rows = (slice_rows + kTileRows - 1) / kTileRows * kTileRows;
    const int p_tiles = rows / kTileRows < kMaxTiles ? rows / kTileRows : kMaxTiles;  // tiles per sub-slice
    TcSmem L;
    int off = 0;
    L.ring = off;
    off += stages * kTcTileBytes;
    L.pbuf = off;
    off += p_tiles * tc_ptile_bytes(G) + 1024;
    L.qbuf = off;
    off += 2 * tc_qbuf_bytes(G);
    L.wsm = off;
    off += rows * 4;  // scaled write score of every slot of the slice
    L.list = off;     // slots the update rule rewrites this token, in no particular order
    off += rows * 2;
    off = (off + 15) & ~15;
    L.lww = off;      // write weights of the first kLwwCap listed slots (the update is applied one unit late)
    off += kLwwCap * 4;
    L.lostage = off;  // staged copies of up to lo_cap of those rows: value plane rows, then residual rows
    off += 2 * lo_cap * 256;
    L.red = off;
    off += 4 * 32 * 4;  // per softmax warp: 16 partial maxima / sums, 16 partial appended-slot scores / overlaps
    L.stat = off;  // m[16], l[16], wd[16], ev[16], alpha[16], abort, tmem address, list count
    off += 512;
    L.vtb = off;   // eta_t * wv_t as floats: the in-ring rewrite of whole tiles reads it as a broadcast
    off += 128 * 4;
    L.wstat = off;
    off += 2 * kMaxClusterTc * 2 * 4;
    L.merge = off;
    off += (S > 1) ? 2 * (S - 1) * G * (128 + 3) * 4 : 0;
    off = (off + 15) & ~15;
    L.bars = off;
    off += (2 * stages + 3 * kMaxTiles + 2 + 1 + 2 + 2 + 1) * 8;
    L.total = ((off + 127) & ~127) + 1024;  // + slack to align the ring to 1024 bytes
    return L;
}

// N = 8 or 16 consecutive columns of this thread's tensor-memory lane
template <int N>
__device__ __forceinline__ void tmem_ld_rows(uint32_t taddr, float* x) {
    if constexpr (N == 8) {
        tmem_ld8(taddr, x);
    } else {
        tmem_ld16(taddr, x);
    }
}
template <int N>
__device__ __forceinline__ void tmem_st_rows(uint32_t taddr, const float* x) {
    tmem_st8(taddr, x);
    if constexpr (N == 16) tmem_st8(taddr + 8, x + 8);
}

__device__ __forceinline__ void s_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kSThreads) : "memory"); }

// The update rule on 16 bytes (8 elements) of one row, MV_t = MV_{t-1} + ww * (eta_t wv_t): the staged value and
// residual chunks give MV_{t-1}, the sum is split again into a bfloat16 value and a bfloat16 residual and
// stored to the two planes.
__device__ __forceinline__ void rewrite_chunk(const unsigned char* staged_hi, const unsigned char* staged_lo, char* dst_hi,
                                              char* dst_lo, float ww, const float* vtv) {
    float x[8], lo[8], nv[8], hf[8];
    Chunk<__nv_bfloat16>::unpack(*reinterpret_cast<const uint4*>(staged_hi), x);
    Chunk<__nv_bfloat16>::unpack(*reinterpret_cast<const uint4*>(staged_lo), lo);
#pragma unroll
    for (int e = 0; e < 8; ++e) nv[e] = fmaf(ww, vtv[e], x[e] + lo[e]);
    const uint4 hi_new = Chunk<__nv_bfloat16>::pack(nv);
    Chunk<__nv_bfloat16>::unpack(hi_new, hf);
#pragma unroll
    for (int e = 0; e < 8; ++e) nv[e] -= hf[e];
    *reinterpret_cast<uint4*>(dst_hi) = hi_new;
    *reinterpret_cast<uint4*>(dst_lo) = Chunk<__nv_bfloat16>::pack(nv);
}

// kSmall: units of at most kSmallTiles tiles, one CTA per unit, two CTAs resident per SM (half the tensor memory,
// a two-stage ring each): a unit of a few tiles is a chain of barriers and latencies in the softmax warps, and two
// CTAs' chains hide each other.
template <int G, bool kSmall>
__global__ void __launch_bounds__(kTcThreads, kSmall ? 2 : 1)
decode_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                 const __grid_constant__ CUtensorMap tmLo, const TcArgs a) {
    constexpr int D = 128;
    constexpr int ROW_BYTES = 256;
    constexpr int NR = tc_rows(G);                 // operand rows kept: read heads, write query, zero rows
    constexpr int kQHalf = NR * 128, kPHalf = NR * 128;  // bytes between the two 64-column halves
    constexpr int kQBufBytes = tc_qbuf_bytes(G), kPTileBytes = tc_ptile_bytes(G);
    constexpr int kOCol = tc_ocol(kSmall), kTmemCols = tc_tmem_cols(kSmall);
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int S = a.S;
    const int NST = a.stages;
    const int kLoCap = a.lo_cap;
    const TcSmem L = tc_smem(NST, G, S, a.slice_rows, kLoCap);
    unsigned char* ring = smem + L.ring;
    unsigned char* pbuf = smem + L.pbuf;
    unsigned char* qbuf = smem + L.qbuf;
    float* wsm = reinterpret_cast<float*>(smem + L.wsm);
    unsigned short* list = reinterpret_cast<unsigned short*>(smem + L.list);
    float* lww = reinterpret_cast<float*>(smem + L.lww);
    unsigned char* histage = smem + L.lostage;
    unsigned char* lostage = histage + kLoCap * ROW_BYTES;
    float* red = reinterpret_cast<float*>(smem + L.red);
    float* st_m = reinterpret_cast<float*>(smem + L.stat);
    float* st_l = st_m + 16;
    float* st_wd = st_m + 32;
    float* st_ev = st_m + 48;
    float* st_alpha = st_m + 64;  // per head: exp(old maximum - new maximum) of the current sub-slice
    volatile int* abort_flag = reinterpret_cast<volatile int*>(st_m + 80);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(st_m + 81);
    int* lo_count = reinterpret_cast<int*>(st_m + 82);
    float* wstat = reinterpret_cast<float*>(smem + L.wstat);
    float* merge = reinterpret_cast<float*>(smem + L.merge);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L.bars);
    uint64_t* empty = full + NST;
    uint64_t* sready = empty + NST;         // [kMaxTiles]: score tile t of the current unit is complete
    uint64_t* pready = sready + kMaxTiles;  // [kMaxTiles]: P operand of tile t of the current unit is written
    uint64_t* qready = pready + kMaxTiles;  // [2]
    uint64_t* oready = qready + 2;
    uint64_t* xbar = oready + 1;            // [2]
    uint64_t* mbar = xbar + 2;              // [2]
    uint64_t* subfree = mbar + 2;           // the score tiles of a sub-slice have been consumed (128 arrivals)
    uint64_t* vdone = subfree + 1;          // [kMaxTiles]: the MMAs that read MV tile t are complete (in-ring rewrite only)
    float* vtb = reinterpret_cast<float*>(smem + L.vtb);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const int rank = (S > 1) ? (int)cluster_ctarank() : 0;
    const int cid = blockIdx.x / S;
    const int ncl = gridDim.x / S;

    const int slice_start = rank * a.slice_rows;
    const int n_slice = max(0, min(a.slice_rows, a.C - slice_start));
    const int n_stream = max(0, min(a.len - slice_start, n_slice));
    const bool has_virtual = (a.len < a.C) && (a.len >= slice_start) && (a.len < slice_start + n_slice);
    const int nt = (n_stream + kTileRows - 1) / kTileRows;   // tiles of the slice
    const int n_sub = (nt + kMaxTiles - 1) / kMaxTiles;       // sub-slices of up to kMaxTiles tiles
    // Every slot rewritten (BCT_FLAG_DENSE_WRITE) and the slice scored in one go: the residual tiles travel through
    // the ring behind their value tiles, the softmax warps rebuild both in place once the tile's products are
    // complete, and the stages go home as TMA stores (no row is read twice, nothing is staged).
    const bool ring_rewrite = !kSmall && a.dense && a.do_write && n_sub == 1;

    if (tid == 0) {
        for (int i = 0; i < NST; ++i) {
            mbar_init(&full[i], 1);
            mbar_init(&empty[i], 1);  // the MMA commit alone frees a stage
        }
        for (int i = 0; i < kMaxTiles; ++i) {
            mbar_init(&sready[i], 1);
            mbar_init(&pready[i], kSThreads);
        }
        mbar_init(&qready[0], kSThreads);
        mbar_init(&qready[1], kSThreads);
        mbar_init(oready, 1);
        mbar_init(subfree, kSThreads);
        for (int i = 0; i < kMaxTiles; ++i) mbar_init(&vdone[i], 1);
        mbar_init(&xbar[0], S);
        mbar_init(&xbar[1], S);
        mbar_init(&mbar[0], kSThreads * (S > 1 ? S - 1 : 1));
        mbar_init(&mbar[1], kSThreads * (S > 1 ? S - 1 : 1));
        *abort_flag = 0;
        *lo_count = 0;
        fence_mbar_init_cluster();
    }
    // zero the operands: rows G..7 of P and rows above the write query of Q stay zero for good,
    // and so do the dummy rows behind them that the N = 16 instruction shape reads
    for (int i = tid; i < 2 * kQBufBytes / 16; i += kTcThreads) reinterpret_cast<uint4*>(qbuf)[i] = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < (L.qbuf - L.pbuf) / 16; i += kTcThreads)
        reinterpret_cast<uint4*>(pbuf)[i] = make_uint4(0, 0, 0, 0);
    if (warp == 5) tmem_alloc(tmem_slot, kTmemCols);
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (S > 1) {
        cluster_arrive();
        cluster_wait();
    }

    if (warp == 4) {
        // =========================== producer ===========================
        if (lane == 0) {
            int stage = 0;        // ring position without divisions: this thread has nothing to hide their latency behind
            uint32_t rph = 0;     // parity of the ring pass
            bool first_pass = true;
            bool ok = true;
            for (int u = cid; u < a.U && ok; u += ncl) {
                for (int ph = 0; ph < 2 * n_sub && ok; ++ph) {  // per sub-slice: its MK tiles, then its MV tiles
                    const CUtensorMap* map = (ph & 1) == 0 ? &tmK : &tmV;
                    const int t_begin = (ph >> 1) * kMaxTiles, t_end = min(nt, t_begin + kMaxTiles);
                    // (with the in-ring rewrite every MV tile is followed by its residual tile)
                    const int per_tile = ((ph & 1) && ring_rewrite) ? 2 : 1;
                    for (int item = t_begin * per_tile; item < t_end * per_tile && ok; ++item) {
                        const int t = item / per_tile;
                        const CUtensorMap* m = (per_tile == 2 && (item & 1)) ? &tmLo : map;
                        if (!first_pass && !mbar_wait_abortable(&empty[stage], rph ^ 1u, abort_flag)) {
                            report_timeout(a.status, 11);
                            *abort_flag = 1;
                            ok = false;
                            break;
                        }
                        unsigned char* dst = ring + (size_t)stage * kTcTileBytes;
                        mbar_arrive_expect_tx(&full[stage], kTcTileBytes);
                        tma_load_3d(dst, m, 0, slice_start + t * kTileRows, u, &full[stage]);
                        tma_load_3d(dst + kHalfBytes, m, 64, slice_start + t * kTileRows, u, &full[stage]);
                        if (++stage == NST) {
                            stage = 0;
                            rph ^= 1u;
                            first_pass = false;
                        }
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 5) {
        // =========================== MMA issuer ===========================
        if (lane == 0) {
            constexpr uint32_t idesc_s = instr_desc(false);
            constexpr uint32_t idesc_o = instr_desc(true);
            uint32_t sp = 0, nsf = 0;  // sub-slices so far, sub-slice hand-overs so far
            int stage = 0;             // ring position and the parity of its pass
            uint32_t rph = 0;
            // descriptors at shared address 0: the address field is added per use (addresses stay below 256 KiB)
            const uint64_t dk0 = smem_desc(0, 16, 1024), dmn0 = smem_desc(0, kHalfBytes, 1024);
            int it = 0;
            for (int u = cid; u < a.U; u += ncl, ++it) {
                if (!mbar_wait_abortable(&qready[it & 1], (it >> 1) & 1, abort_flag)) {
                    report_timeout(a.status, 12);
                    *abort_flag = 1;
                }
                tc_fence_after();
                const uint32_t qaddr = smem_u32(qbuf + (it & 1) * kQBufBytes);
                for (int sub = 0; sub < n_sub; ++sub, ++sp) {
                    const int t_begin = sub * kMaxTiles, t_end = min(nt, t_begin + kMaxTiles);
                    if (sub > 0) {  // the previous sub-slice's score tiles must have been consumed
                        if (!mbar_wait_abortable(subfree, nsf & 1, abort_flag)) {
                            report_timeout(a.status, 22);
                            *abort_flag = 1;
                        }
                        ++nsf;
                        tc_fence_after();
                    }
                    for (int t = t_begin; t < t_end; ++t) {  // scores: A = K tile (K-major), B = Q (K-major)
                        if (!mbar_wait_abortable(&full[stage], rph, abort_flag)) {
                            report_timeout(a.status, 13);
                            *abort_flag = 1;
                        }
                        tc_fence_after();
                        const uint32_t taddr = smem_u32(ring + (size_t)stage * kTcTileBytes);
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {
                            const uint64_t ad = desc_at(dk0, taddr + (kk >> 2) * kHalfBytes + (kk & 3) * 32);
                            const uint64_t bd = desc_at(dk0, qaddr + (kk >> 2) * kQHalf + (kk & 3) * 32);
                            umma_bf16(tmem_base + (t - t_begin) * kScoreCols, ad, bd, idesc_s, kk > 0);
                        }
                        umma_commit(&sready[t - t_begin]);
                        umma_commit(&empty[stage]);
                        if (++stage == NST) {
                            stage = 0;
                            rph ^= 1u;
                        }
                    }
                    for (int t = t_begin; t < t_end; ++t) {  // outputs: A = V tile (MN-major), B = P (K-major)
                        if (!mbar_wait_abortable(&pready[t - t_begin], sp & 1, abort_flag)) {
                            report_timeout(a.status, 14);
                            *abort_flag = 1;
                        }
                        if (!mbar_wait_abortable(&full[stage], rph, abort_flag)) {
                            report_timeout(a.status, 15);
                            *abort_flag = 1;
                        }
                        tc_fence_after();
                        const uint32_t taddr = smem_u32(ring + (size_t)stage * kTcTileBytes);
                        const uint32_t paddr = smem_u32(pbuf + (t - t_begin) * kPTileBytes);
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {  // 16 slots per step
                            const uint64_t ad = desc_at(dmn0, taddr + kk * 2048);
                            const uint64_t bd = desc_at(dk0, paddr + (kk >> 2) * kPHalf + (kk & 3) * 32);
                            umma_bf16(tmem_base + kOCol, ad, bd, idesc_o, (t > 0) || (kk > 0));
                        }
                        if (ring_rewrite) {
                            // the softmax warps rebuild the tile in its stage and release it; the residual tile's
                            // stage is theirs alone
                            umma_commit(&vdone[t - t_begin]);
                            if (++stage == NST) {
                                stage = 0;
                                rph ^= 1u;
                            }
                        } else {
                            umma_commit(&empty[stage]);
                        }
                        if (++stage == NST) {
                            stage = 0;
                            rph ^= 1u;
                        }
                    }
                    umma_commit(oready);  // every V tile of the sub-slice has been read
                }
            }
        }
        __syncwarp();
    } else {
        // =========================== softmax / epilogue / update warps ===========================
        const int r = tid;  // tensor-memory lane: slot row of a score tile, d of the output
        const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);

        // Q operand of a unit: rows 0..G-1 its read queries, row G its write query (128-byte swizzle).
        // The words are fetched from global memory at the start of the previous unit's turn and put in
        // place when that unit's score tiles have been consumed: their latency would otherwise sit in
        // every unit's chain (about 1 us of the 6 us a unit of 256 slots takes).
        constexpr int kQWords = (NR + 7) / 8;  // 16-byte words of the operand per thread
        auto load_q = [&](int u, uint4* w) {
            const int b = u / a.Hkv;
            const int h_kv = u - b * a.Hkv;
            const int c = tid & 15;
#pragma unroll
            for (int i = 0; i < kQWords; ++i) {
                const int h = (tid >> 4) + i * (kSThreads / 16);
                if (h <= G) {
                    const char* src = (h < G) ? a.q + ((size_t)b * a.q_bs + (size_t)h_kv * G * D) * 2 + (size_t)h * ROW_BYTES
                                              : a.k + ((size_t)b * a.kv_bs + (size_t)h_kv * D) * 2;
                    w[i] = *reinterpret_cast<const uint4*>(src + c * 16);
                }
            }
        };
        auto store_q = [&](int buf, const uint4* w) {
            const int c = tid & 15;
#pragma unroll
            for (int i = 0; i < kQWords; ++i) {
                const int h = (tid >> 4) + i * (kSThreads / 16);
                if (h <= G) {
                    unsigned char* dst = qbuf + buf * kQBufBytes + (c >> 3) * kQHalf + h * 128 + (((c & 7) ^ (h & 7)) * 16);
                    *reinterpret_cast<uint4*>(dst) = w[i];
                }
            }
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(&qready[buf]);
        };
        uint4 qnext[kQWords];
        if (cid < a.U) {
            load_q(cid, qnext);
            store_q(0, qnext);
        }

        // Staging of the rows the update rule rewrites: copies of their value and residual rows arrive in shared
        // memory by 16-byte asynchronous copies, so that no global-memory latency is left for the update.
        const int c16 = tid & 15;  // 16-byte chunk of a 256-byte row
        auto stage_rows = [&](size_t uoff, int base, int n, int sbase) {
            for (int i = tid >> 4; i < n; i += kSThreads / 16) {
                const size_t goff = uoff + (size_t)(slice_start + list[base + i]) * ROW_BYTES + c16 * 16;
                cp_async16(histage + (sbase + i) * ROW_BYTES + c16 * 16, a.vhi + goff);
                cp_async16(lostage + (sbase + i) * ROW_BYTES + c16 * 16, a.vlo + goff);
            }
            cp_async_commit();
        };
        // The update rule MV_t = MV_{t-1} + ww_t^T . wv_t on listed rows [base, base + n), staged from row sbase
        // of the staging area on; their weights come from lww (kept across units) or from the scaled scores.
        auto rewrite_rows = [&](size_t uoff, int base, int n, int sbase, const float* vtv, bool from_lww, float wmax, float wfac) {
            for (int i = tid >> 4; i < n; i += kSThreads / 16) {
                const int row = list[base + i];
                const float ww = from_lww ? lww[base + i] : __expf(wsm[row] - wmax) * wfac;
                const size_t goff = uoff + (size_t)(slice_start + row) * ROW_BYTES + c16 * 16;
                rewrite_chunk(histage + (sbase + i) * ROW_BYTES + c16 * 16, lostage + (sbase + i) * ROW_BYTES + c16 * 16,
                              a.vhi + goff, a.vlo + goff, ww, vtv);
            }
        };
        // A unit's deferred update: rounds of kLoCap staged rows (weights kept in lww), whose first round has been
        // in flight since that unit's epilogue.
        auto apply_update = [&](int n_rows, size_t uoff, const float* vtv) {
            for (int base = 0; base < n_rows; base += kLoCap) {
                const int n = min(n_rows - base, kLoCap);
                if (base > 0) {
                    s_sync();  // the previous round's staged rows have been consumed
                    stage_rows(uoff, base, n, 0);
                }
                cp_async_wait_all();
                s_sync();  // every thread's staged chunks have landed
                rewrite_rows(uoff, base, n, 0, vtv, true, 0.f, 0.f);
            }
        };
        unsigned long long rows_stored = 0;  // thread 0: MV rows this CTA has rewritten

        int it = 0;
        uint32_t sp = 0;  // sub-slices processed so far (phase of the per-tile barriers)
        // update of the previous unit, applied during this unit's turn: rows listed, plane offset, v_t * eta_t
        int pend_n = 0;
        size_t pend_off = 0;
        float pend_vt[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        const int n_sub_rows = max(n_sub, 1);  // a unit with no tile still has its appended slot to look after
        for (int u = cid; u < a.U; u += ncl, ++it) {
            const int b = u / a.Hkv;
            const int h_kv = u - b * a.Hkv;
            const size_t q_off = ((size_t)b * a.q_bs + (size_t)h_kv * G * D) * 2;
            const size_t kv_off = ((size_t)b * a.kv_bs + (size_t)h_kv * D) * 2;
            // step size of this token's write: MV_t = MV_{t-1} + eta_t ww_t^T wv_t
            const float eta_u = (a.eta != nullptr && a.do_write) ? a.eta[(size_t)b * a.eta_bs + h_kv] : 1.f;
            const size_t unit_off = (size_t)u * a.C * ROW_BYTES;
            if (u + ncl < a.U) load_q(u + ncl, qnext);  // the next unit's operand words: used after this unit's pass 2
            // this thread's 16 bytes of v_t for the update, asked for now so that they have arrived by then
            const uint4 vt_raw = a.do_write ? *reinterpret_cast<const uint4*>(a.v + kv_off + (tid & 15) * 16) : make_uint4(0, 0, 0, 0);

            // the appended slot (fill phase) is scored from the step vectors; v_t[d] is also what a read that
            // follows its own write adds
            float vq[G];
            const float kd = has_virtual ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(a.k + kv_off)[r]) : 0.f;
            const float vd = (has_virtual || (a.wtr && a.do_write))
                                 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(a.v + kv_off)[r]) : 0.f;
            const float vd_w = ring_rewrite ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(a.v + kv_off)[r]) : 0.f;
#pragma unroll
            for (int g = 0; g < G; ++g) {
                vq[g] = 0.f;
                if (has_virtual) {
                    const float qd = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(a.q + q_off)[g * D + r]);
                    vq[g] = warp_sum(qd * kd);
                }
            }
            if (tid < NR) {  // running maximum, sum and read-write overlap of the unit, over its sub-slices
                st_m[tid] = kNegBigTc;
                st_l[tid] = 0.f;
                st_wd[tid] = 0.f;
            }

            // A slice longer than the tensor memory can score at once is taken in sub-slices of up to
            // kMaxTiles tiles; maxima, sums and the output accumulator are rescaled from one to the next.
            for (int sub = 0; sub < n_sub_rows; ++sub, ++sp) {
                const int t_begin = sub * kMaxTiles, t_end = min(nt, t_begin + kMaxTiles);
                const bool last_sub = (sub == n_sub_rows - 1);

                // ---- pass 1: row maxima of the raw scores, as the score tiles complete ----
                float mx[NR];
#pragma unroll
                for (int h = 0; h < NR; ++h) mx[h] = kNegBigTc;
                for (int t = t_begin; t < t_end; ++t) {
                    if (!mbar_wait_abortable(&sready[t - t_begin], sp & 1, abort_flag)) {
                        report_timeout(a.status, 16);
                        *abort_flag = 1;
                    }
                    tc_fence_after();
                    float s[NR];
                    tmem_ld_rows<NR>(lane_base + (t - t_begin) * kScoreCols, s);
                    if (t * kTileRows + r < n_stream) {
#pragma unroll
                        for (int h = 0; h < NR; ++h) mx[h] = fmaxf(mx[h], s[h]);
                    }
                }
#pragma unroll
                for (int h = 0; h < NR; ++h) {
                    mx[h] = warp_max(mx[h]);
                    if (lane == 0) red[warp * 32 + h] = mx[h];
                    if (lane == 0 && h < G) red[warp * 32 + 16 + h] = vq[h];
                }
                s_sync();
                if (tid < NR) {
                    const float scale = (tid < G) ? a.read_scale : a.write_scale;
                    float m = fmaxf(fmaxf(red[tid], red[32 + tid]), fmaxf(red[64 + tid], red[96 + tid]));
                    m = (m <= kNegBigTc) ? kNegBigTc : m * scale;
                    if (last_sub && has_virtual && tid < G) {
                        const float vs = (red[16 + tid] + red[48 + tid] + red[80 + tid] + red[112 + tid]) * a.read_scale;
                        st_ev[tid] = vs;  // scaled score of the appended slot, turned into a numerator below
                        m = fmaxf(m, vs);
                    }
                    const float m_old = st_m[tid];
                    const float m_new = fmaxf(m_old, m);
                    st_alpha[tid] = (m_old <= kNegBigTc) ? 0.f : __expf(m_old - m_new);
                    st_m[tid] = m_new;
                }
                s_sync();

                // ---- the outputs accumulated so far refer to the old maxima: rescale them in tensor memory ----
                if (sub > 0) {
                    if (!mbar_wait_abortable(oready, (sp - 1) & 1, abort_flag)) {
                        report_timeout(a.status, 23);
                        *abort_flag = 1;
                    }
                    tc_fence_after();
                    float o[NR];
                    tmem_ld_rows<NR>(lane_base + kOCol, o);
#pragma unroll
                    for (int h = 0; h < NR; ++h) o[h] *= st_alpha[h];
                    tmem_st_rows<NR>(lane_base + kOCol, o);
                    tc_fence_before();
                }

                // ---- pass 2: numerators, row sums, P operand (bfloat16, swizzled), scaled write scores ----
                float sum[NR];
                float wdacc[G];
#pragma unroll
                for (int h = 0; h < NR; ++h) sum[h] = 0.f;
#pragma unroll
                for (int g = 0; g < G; ++g) wdacc[g] = 0.f;
                for (int t = t_begin; t < t_end; ++t) {
                    float s[NR];
                    tmem_ld_rows<NR>(lane_base + (t - t_begin) * kScoreCols, s);
                    const bool valid = t * kTileRows + r < n_stream;
                    float e[NR];
#pragma unroll
                    for (int h = 0; h < NR; ++h) {
                        const float scale = (h < G) ? a.read_scale : a.write_scale;
                        e[h] = (valid && h <= G) ? __expf(s[h] * scale - st_m[h]) : 0.f;
                        sum[h] += e[h];
                    }
                    unsigned char* prow = pbuf + (t - t_begin) * kPTileBytes + (r >> 6) * kPHalf + (r & 7) * 2;
                    const int c8 = (r & 63) >> 3;
#pragma unroll
                    for (int h = 0; h < G; ++h)  // rows G..7 of the operand stay zero
                        *reinterpret_cast<__nv_bfloat16*>(prow + h * 128 + ((c8 ^ (h & 7)) * 16)) = __float2bfloat16_rn(e[h]);
                    wsm[t * kTileRows + r] = valid ? s[G] * a.write_scale : kNegBigTc;
#pragma unroll
                    for (int g = 0; g < G; ++g) wdacc[g] = fmaf(e[g], e[G], wdacc[g]);
                    fence_proxy_async_smem();
                    tc_fence_before();
                    mbar_arrive(&pready[t - t_begin]);  // the V tile's MMAs may go as soon as its weights are in place
                }
                if (last_sub) {
                    // the next unit's scores may start as soon as this unit's V tiles are through
                    if (u + ncl < a.U) store_q((it + 1) & 1, qnext);
                } else {
                    tc_fence_before();
                    mbar_arrive(subfree);  // this sub-slice's score tiles may be overwritten
                }

#pragma unroll
                for (int h = 0; h < NR; ++h) {
                    sum[h] = warp_sum(sum[h]);
                    if (lane == 0) red[warp * 32 + h] = sum[h];
                }
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    wdacc[g] = warp_sum(wdacc[g]);
                    if (lane == 0) red[warp * 32 + 16 + g] = wdacc[g];
                }
                s_sync();
                if (tid < NR) {
                    float l = red[tid] + red[32 + tid] + red[64 + tid] + red[96 + tid];
                    if (last_sub && has_virtual && tid < G) {
                        const float ev = __expf(st_ev[tid] - st_m[tid]);
                        st_ev[tid] = ev;
                        l += ev;
                    }
                    st_l[tid] = st_l[tid] * st_alpha[tid] + l;
                    st_wd[tid] = st_wd[tid] * st_alpha[tid] * st_alpha[G] +
                                 (red[16 + tid] + red[48 + tid] + red[80 + tid] + red[112 + tid]);
                }
                s_sync();
            }

            // ---- write weights are normalised over ALL C slots: exchange across the cluster ----
            float wfac = 0.f;
            if (a.do_write) {
                if (S > 1) {
                    float* ws = wstat + (it & 1) * kMaxClusterTc * 2;
                    if (tid == 0) {
                        for (int rr = 0; rr < S; ++rr) {
                            const uint32_t dst = map_to_rank(ws + 2 * rank, rr);
                            st_cluster_f32(dst, st_m[G]);
                            st_cluster_f32(dst + 4, st_l[G]);
                            mbar_arrive_remote(map_to_rank(&xbar[it & 1], rr));
                        }
                    }
                    if (!mbar_wait_abortable<true>(&xbar[it & 1], (it >> 1) & 1, abort_flag)) {
                        report_timeout(a.status, 17);
                        *abort_flag = 1;
                    }
                    float M = kNegBigTc;
                    for (int rr = 0; rr < S; ++rr) M = fmaxf(M, ws[2 * rr]);
                    float Ls = 0.f;
                    for (int rr = 0; rr < S; ++rr) Ls += ws[2 * rr + 1] * __expf(ws[2 * rr] - M);
                    wfac = __expf(st_m[G] - M) / Ls;
                } else {
                    wfac = 1.f / st_l[G];
                }
            }

            // ---- list the slots the rule rewrites and stage copies of their value and residual rows (stage_rows),
            // ---- so that no global-memory latency is left for the update ----
            // The previous unit's rows first: their staged copies had this unit's whole softmax to arrive,
            // and this unit's V tiles are being multiplied meanwhile.  (Units are independent memories.)
            if (pend_n > 0) {
                apply_update(pend_n, pend_off, pend_vt);
                pend_n = 0;
                s_sync();  // the list and the staging rows are free for this unit
                if (tid == 0) *lo_count = 0;
                s_sync();
            }
            if (ring_rewrite) {
                // Every slot is rewritten: tile by tile in the ring stages the value and residual tiles arrived in,
                // as soon as the products that read the value tile are complete; the stages go home as TMA stores.
                // Thread r holds row r of the tile; eta_t * wv_t is read from shared memory as a broadcast.
                vtb[r] = vd_w * eta_u;
                s_sync();
                const uint32_t item0 = (uint32_t)it * (3u * (uint32_t)nt) + (uint32_t)nt;  // ring items so far: 3 nt per unit
                const int sw7 = r & 7;
                for (int t = 0; t < nt; ++t) {
                    const uint32_t ih = item0 + 2u * t, il = ih + 1u;
                    const int sh = (int)(ih % (uint32_t)NST), sl = (int)(il % (uint32_t)NST);
                    if (!mbar_wait_abortable(&vdone[t], (sp - 1) & 1, abort_flag) ||
                        !mbar_wait_abortable(&full[sh], (ih / (uint32_t)NST) & 1u, abort_flag) ||
                        !mbar_wait_abortable(&full[sl], (il / (uint32_t)NST) & 1u, abort_flag)) {
                        report_timeout(a.status, 24);
                        *abort_flag = 1;
                    }
                    const int row = t * kTileRows + r;
                    const float ww = (row < n_stream) ? __expf(wsm[row] - st_m[G]) * wfac : 0.f;
                    unsigned char* th = ring + (size_t)sh * kTcTileBytes + r * 128;
                    unsigned char* tl = ring + (size_t)sl * kTcTileBytes + r * 128;
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
#pragma unroll 2
                        for (int c = 0; c < 8; ++c) {
                            const int off = hh * kHalfBytes + ((c ^ sw7) * 16);
                            const float4 va = *reinterpret_cast<const float4*>(vtb + hh * 64 + c * 8);
                            const float4 vb = *reinterpret_cast<const float4*>(vtb + hh * 64 + c * 8 + 4);
                            const float v8[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
                            rewrite_chunk(th + off, tl + off, reinterpret_cast<char*>(th + off), reinterpret_cast<char*>(tl + off),
                                          ww, v8);
                        }
                    }
                    fence_proxy_async_smem();
                    s_sync();  // the whole tile has been rebuilt
                    if (tid == 0) {
                        const int y = slice_start + t * kTileRows;  // rows past C are clipped by the store
                        unsigned char* bh = ring + (size_t)sh * kTcTileBytes;
                        unsigned char* bl = ring + (size_t)sl * kTcTileBytes;
                        tma_store_3d(&tmV, 0, y, u, bh);
                        tma_store_3d(&tmV, 64, y, u, bh + kHalfBytes);
                        tma_store_3d(&tmLo, 0, y, u, bl);
                        tma_store_3d(&tmLo, 64, y, u, bl + kHalfBytes);
                        bulk_commit();
                        bulk_wait_read();  // the stages have been read out: they may be refilled
                        mbar_arrive(&empty[sh]);
                        mbar_arrive(&empty[sl]);
                    }
                }
                if (tid == 0) rows_stored += (unsigned long long)n_stream;
            }
            int n_touched = 0;
            if (a.do_write && !ring_rewrite) {
                for (int t = 0; t < nt; ++t) {
                    const int row = t * kTileRows + r;
                    const float ww = (row < n_stream) ? __expf(wsm[row] - st_m[G]) * wfac : 0.f;
                    if (row < n_stream && (a.dense || ww >= a.write_eps)) {
                        const int idx = atomicAdd(lo_count, 1);
                        list[idx] = (unsigned short)row;
                        if (idx < kLwwCap) lww[idx] = ww;
                    }
                }
                s_sync();
                n_touched = *lo_count;
                // (a unit that rewrites more rows than lww keeps goes in double-buffered half rounds, below)
                stage_rows(unit_off, 0, min(n_touched, n_touched > kLwwCap ? kLoCap / 2 : kLoCap), 0);
                if (tid == 0) rows_stored += (unsigned long long)n_touched;
            }

            // ---- epilogue: O[d][g] from tensor memory once every V tile has been read ----
            if (nt > 0 && !mbar_wait_abortable(oready, (sp - 1) & 1, abort_flag)) {
                report_timeout(a.status, 19);
                *abort_flag = 1;
            }
            tc_fence_after();
            float o[NR];
            if (nt > 0) {
                tmem_ld_rows<NR>(lane_base + kOCol, o);
            } else {
#pragma unroll
                for (int h = 0; h < NR; ++h) o[h] = 0.f;
            }
            tc_fence_before();
            if (has_virtual) {
#pragma unroll
                for (int g = 0; g < G; ++g) o[g] = fmaf(st_ev[g], vd, o[g]);
            }
            const bool add_own = a.wtr && a.do_write;
            if (S == 1) {
                if (a.out != nullptr && !*abort_flag) {
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const float inv = 1.f / st_l[g];
                        float val = o[g] * inv;
                        if (add_own) val = fmaf(st_wd[g] * inv * wfac, vd * eta_u, val);
                        if (a.out_f32)
                            reinterpret_cast<float*>(a.out + q_off * 2)[g * D + r] = val;
                        else
                            reinterpret_cast<__nv_bfloat16*>(a.out + q_off)[g * D + r] = __float2bfloat16_rn(val);
                    }
                }
            } else {
                float* mg = merge + (size_t)(it & 1) * (S - 1) * G * (D + 3);
                if (rank != 0) {
                    float* dst0 = mg + (size_t)(rank - 1) * G * (D + 3);
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        st_cluster_f32(map_to_rank(dst0 + g * (D + 3) + r, 0), o[g]);
                        if (r == 0) {
                            st_cluster_f32(map_to_rank(dst0 + g * (D + 3) + D, 0), st_wd[g] * wfac);
                            st_cluster_f32(map_to_rank(dst0 + g * (D + 3) + D + 1, 0), st_m[g]);
                            st_cluster_f32(map_to_rank(dst0 + g * (D + 3) + D + 2, 0), st_l[g]);
                        }
                    }
                    mbar_arrive_remote(map_to_rank(&mbar[it & 1], 0));
                } else {
                    if (!mbar_wait_abortable<true>(&mbar[it & 1], (it >> 1) & 1, abort_flag)) {
                        report_timeout(a.status, 20);
                        *abort_flag = 1;
                    }
                    if (a.out != nullptr && !*abort_flag) {
#pragma unroll
                        for (int g = 0; g < G; ++g) {
                            float M = st_m[g];
                            for (int rr = 1; rr < S; ++rr) M = fmaxf(M, mg[((rr - 1) * G + g) * (D + 3) + D + 1]);
                            const float f0 = __expf(st_m[g] - M);
                            float num = o[g] * f0, own = st_wd[g] * wfac * f0, den = st_l[g] * f0;
                            for (int rr = 1; rr < S; ++rr) {
                                const float* mr = mg + ((rr - 1) * G + g) * (D + 3);
                                const float f = __expf(mr[D + 1] - M);
                                num = fmaf(mr[r], f, num);
                                own = fmaf(mr[D], f, own);
                                den = fmaf(mr[D + 2], f, den);
                            }
                            float val = num / den;
                            if (add_own) val = fmaf(own / den, vd * eta_u, val);
                            if (a.out_f32)
                                reinterpret_cast<float*>(a.out + q_off * 2)[g * D + r] = val;
                            else
                                reinterpret_cast<__nv_bfloat16*>(a.out + q_off)[g * D + r] = __float2bfloat16_rn(val);
                        }
                    }
                }
            }

            // ---- the update: deferred to the next unit's turn (its weights are in lww), unless it rewrites
            // ---- more rows than lww keeps (diffuse write weights): then it is applied here ----
            if (a.do_write && n_touched > 0) {
                float vt[8];
                Chunk<__nv_bfloat16>::unpack(vt_raw, vt);
#pragma unroll
                for (int e = 0; e < 8; ++e) vt[e] *= eta_u;
                if (n_touched <= kLwwCap) {
                    pend_n = n_touched;
                    pend_off = unit_off;
#pragma unroll
                    for (int e = 0; e < 8; ++e) pend_vt[e] = vt[e];
                } else {
                    // Diffuse write weights: most rows of the slice.  Half rounds alternate between the two
                    // halves of the staging area, so that one half round is rewritten while the next arrives.
                    const int hcap = kLoCap / 2;
                    const int n_rounds = (n_touched + hcap - 1) / hcap;
                    for (int rd = 0; rd < n_rounds; ++rd) {
                        const int base = rd * hcap, n = min(n_touched - base, hcap);
                        const int sbase = (rd & 1) * hcap;  // first staging row of this half round
                        if (rd + 1 < n_rounds) {  // ask for the next half round (its half was consumed a round ago)
                            const int nb = base + hcap;
                            stage_rows(unit_off, nb, min(n_touched - nb, hcap), ((rd + 1) & 1) * hcap);
                            cp_async_wait_but_one();
                        } else {
                            cp_async_wait_all();
                        }
                        s_sync();  // this half round's chunks have landed for every thread
                        rewrite_rows(unit_off, base, n, sbase, vt, false, st_m[G], wfac);
                        s_sync();  // the half is free for the round after next
                    }
                }
            }
            if (has_virtual && tid < 16) {  // store the appended slot
                const size_t off = unit_off + (size_t)a.len * ROW_BYTES + tid * 16;
                *reinterpret_cast<uint4*>(a.kplane + off) = *reinterpret_cast<const uint4*>(a.k + kv_off + tid * 16);
                *reinterpret_cast<uint4*>(a.vhi + off) = *reinterpret_cast<const uint4*>(a.v + kv_off + tid * 16);
                *reinterpret_cast<uint4*>(a.vlo + off) = make_uint4(0, 0, 0, 0);
            }
            s_sync();  // st_*, red and wsm are reused by the next unit (the list and the staging rows: after its deferred update)
            if (pend_n == 0 && tid == 0) *lo_count = 0;
        }
        if (pend_n > 0) apply_update(pend_n, pend_off, pend_vt);  // the last unit's rows
        if (ring_rewrite && tid == 0) bulk_wait_all();              // the last tiles' stores have landed
        if (tid == 0 && rows_stored > 0)
            atomicAdd(reinterpret_cast<unsigned long long*>(a.status + kStatusRowsWord), rows_stored);
    }

    tc_fence_before();
    __syncthreads();
    if (S > 1) {  // nobody leaves while a peer may still write its shared memory
        cluster_arrive();
        cluster_wait();
    }
    if (warp == 5) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

using TcKernelFn = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const TcArgs);

TcKernelFn pick_tc(int G, bool small) {
    if (small) {
        switch (G) {
            case 1: return decode_tc_kernel<1, true>;
            case 2: return decode_tc_kernel<2, true>;
            case 3: return decode_tc_kernel<3, true>;
            case 4: return decode_tc_kernel<4, true>;
            case 5: return decode_tc_kernel<5, true>;
            case 6: return decode_tc_kernel<6, true>;
            case 7: return decode_tc_kernel<7, true>;
            default: return nullptr;
        }
    }
    switch (G) {
        case 1: return decode_tc_kernel<1, false>;
        case 2: return decode_tc_kernel<2, false>;
        case 3: return decode_tc_kernel<3, false>;
        case 4: return decode_tc_kernel<4, false>;
        case 5: return decode_tc_kernel<5, false>;
        case 6: return decode_tc_kernel<6, false>;
        case 7: return decode_tc_kernel<7, false>;
        case 8: return decode_tc_kernel<8, false>;
        case 9: return decode_tc_kernel<9, false>;
        case 10: return decode_tc_kernel<10, false>;
        case 11: return decode_tc_kernel<11, false>;
        case 12: return decode_tc_kernel<12, false>;
        case 13: return decode_tc_kernel<13, false>;
        case 14: return decode_tc_kernel<14, false>;
        case 15: return decode_tc_kernel<15, false>;
        default: return nullptr;
    }
}

// [U][C][128] bfloat16 plane as a 3-D tensor (d, slot, unit); boxes of 64 x 128 x 1 with the
// 128-byte swizzle; rows past C read as zeros.
bool make_plane_map(CUtensorMap* map, void* base, int U, int C) {
    TensorMapEncodeFn fn = tensor_map_encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[3] = {128, (cuuint64_t)C, (cuuint64_t)U};
    const cuuint64_t strides[2] = {256, (cuuint64_t)C * 256};
    const cuuint32_t box[3] = {64, (cuuint32_t)kTileRows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// cuTensorMapEncodeTiled through the runtime's driver entry point lookup (no link against libcuda).
TensorMapEncodeFn tensor_map_encode_fn() {
    static TensorMapEncodeFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<TensorMapEncodeFn>(p);
    }
    return fn;
}

bool tc_eligible(const bct_cache* c) {
    const bct_params_t& p = c->p;
    if (p.dtype != BCT_BF16 || p.head_dim != 128 || c->G > 15) return false;
    if (p.flags & BCT_FLAG_PRECISE_READ) return false;
    if (p.capacity < kTileRows || p.capacity > kMaxClusterTc * kMaxSliceRows) return false;
    if (c->plane_bytes < (size_t)1 << 18) return false;  // tiny planes stay on the CUDA-core kernel
    return c->tc_ready != 0;
}

bool tc_prepare(bct_cache* c) {
    c->tc_ready = 0;
    static_assert(sizeof(CUtensorMap) <= sizeof(c->tmap_k), "tensor map storage too small");
    if (c->p.dtype != BCT_BF16 || c->p.head_dim != 128) return false;
    if (!make_plane_map(reinterpret_cast<CUtensorMap*>(c->tmap_k), c->kplane, c->U, c->p.capacity)) return false;
    if (!make_plane_map(reinterpret_cast<CUtensorMap*>(c->tmap_v), c->vhi, c->U, c->p.capacity)) return false;
    if (!make_plane_map(reinterpret_cast<CUtensorMap*>(c->tmap_lo), c->vlo, c->U, c->p.capacity)) return false;
    c->tc_ready = 1;
    return true;
}

int launch_decode_tc(const bct_cache* c, const StepIO& io, int len, int do_write, cudaStream_t stream,
                     cudaError_t* err) {
    const bct_params_t& p = c->p;
    // Cluster size: clusters of 2 tile the whole chip (74 x 2 = 148 SMs), clusters of 4 and 8 only 132
    // and 120 SMs, so a unit is split over at most 2 CTAs and a long slice is taken in sub-slices
    // (up to kMaxSliceRows slots per CTA).  Only when there are too few units to fill the SMs is a unit
    // spread wider.
    int S = 1;
    if (p.capacity > kMaxTiles * kTileRows) S = 2;
    while (S < kMaxClusterTc && (p.capacity + S - 1) / S > kMaxSliceRows) S *= 2;
    // few units: spread each over more SMs, as long as the merge buffer of the wider cluster (it grows with
    // the cluster size times the group size) still leaves room for the smallest ring and staging area
    while (S < kMaxClusterTc && (long long)c->U * S * 2 <= c->sm_count && (p.capacity + 2 * S - 1) / (2 * S) >= kTileRows) {
        const int s2 = 2 * S;
        const int slice2 = ((p.capacity + s2 - 1) / s2 + kTileRows - 1) / kTileRows * kTileRows;
        if (tc_smem(3, c->G, s2, slice2, 32).total > c->smem_optin) break;
        S = s2;
    }
    int slice = (p.capacity + S - 1) / S;
    slice = (slice + kTileRows - 1) / kTileRows * kTileRows;  // whole tiles per CTA
    // Four ring stages and staging rounds of 80 rows where shared memory allows (slices up to 2048
    // slots); longer slices keep more per-slot state and give up staging rows first, then a stage.
    // (A deeper ring for short slices was measured: no gain, the softmax chain of a unit is the limit.)
    int lo_cap = 80;
    int stages = 4;
    // Units of up to 512 slots (4 tiles), more than two of them per SM: two CTAs per SM with a two-stage ring, staging
    // rounds of 32 rows and half the tensor memory each.  Such a unit streams in under 1.5 us and its turn in the
    // softmax warps is a chain of about eight barriers: measured, one CTA per SM left the HBM idle a third of the time.
    // (The in-ring rewrite of BCT_FLAG_DENSE_WRITE keeps the one-CTA form.)
    constexpr int kTwoPerSmLimit = 113 * 1024;  // two CTAs and their reserved kilobyte each within an SM's shared memory
    const bool small = S == 1 && slice <= 4 * kTileRows && c->G <= 7 && c->U > 2 * c->sm_count &&
                       !(p.flags & BCT_FLAG_DENSE_WRITE) && tc_smem(2, c->G, 1, slice, 32).total <= kTwoPerSmLimit;
    if (small) {
        stages = 2;
        lo_cap = 32;
    }
    TcKernelFn fn = pick_tc(c->G, small);
    if (fn == nullptr) {
        *err = cudaErrorInvalidConfiguration;
        return -1;
    }
    while (tc_smem(stages, c->G, S, slice, lo_cap).total > c->smem_optin && (stages > 3 || lo_cap > 32)) {
        if (stages > 4 || (stages > 3 && lo_cap <= 48))
            --stages;
        else
            lo_cap -= 16;
    }
    const int smem = tc_smem(stages, c->G, S, slice, lo_cap).total;
    if (smem > c->smem_optin) {
        *err = cudaErrorInvalidConfiguration;
        return -1;
    }

    TcArgs a;
    a.vhi = c->vhi;
    a.vlo = c->vlo;
    a.kplane = c->kplane;
    a.q = static_cast<const char*>(io.q);
    a.k = static_cast<const char*>(io.k);
    a.v = static_cast<const char*>(io.v);
    a.out = static_cast<char*>(io.out);
    a.status = c->status;
    a.q_bs = io.q_batch_stride;
    a.kv_bs = io.kv_batch_stride;
    a.eta = io.eta;
    a.eta_bs = io.eta_batch_stride;
    a.C = p.capacity;
    a.len = len;
    a.slice_rows = slice;
    a.S = S;
    a.Hkv = p.n_kv_heads;
    a.U = c->U;
    a.stages = stages;
    a.lo_cap = lo_cap;
    a.do_write = (len == p.capacity) && do_write;
    a.wtr = (p.flags & BCT_FLAG_WRITE_THEN_READ) ? 1 : 0;
    a.dense = (p.flags & BCT_FLAG_DENSE_WRITE) ? 1 : 0;
    a.out_f32 = (p.flags & BCT_FLAG_OUT_F32) ? 1 : 0;
    a.read_scale = p.read_scale;
    a.write_scale = p.write_scale;
    a.write_eps = p.write_eps;

    // Per (device, group size): the shared-memory limit already set for the kernel, and the last cluster
    // occupancy answer.  Both are runtime calls that a step of tens of microseconds would notice.
    struct Seen {
        int smem_set, occ_S, occ_smem, occ_active;
    };
    // (The table is the only state shared between handles: guarded, and held for the launch itself so that
    // two threads cannot interleave the attribute update and the launches that rely on it.)
    static std::mutex seen_mu;
    static Seen seen[64][2][16] = {};
    std::lock_guard<std::mutex> seen_lock(seen_mu);
    Seen local = {};
    Seen& sn = (c->device >= 0 && c->device < 64) ? seen[c->device][small ? 1 : 0][c->G] : local;
    if (sn.smem_set < smem) {
        *err = cudaFuncSetAttribute(reinterpret_cast<const void*>(fn), cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (*err != cudaSuccess) return -1;
        if (small) {  // the largest shared-memory carve-out, or the SM would be configured for one CTA of this size
            *err = cudaFuncSetAttribute(reinterpret_cast<const void*>(fn), cudaFuncAttributePreferredSharedMemoryCarveout,
                                        cudaSharedmemCarveoutMaxShared);
            if (*err != cudaSuccess) return -1;
        }
        sn.smem_set = smem;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kTcThreads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)S;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n_clusters = c->sm_count / S;
    if (S > 1) {
        cfg.gridDim = dim3((unsigned)(S * (c->sm_count / S)), 1, 1);
        int active = 0;
        if (sn.occ_S == S && sn.occ_smem == smem) {
            active = sn.occ_active;
        } else {
            *err = cudaOccupancyMaxActiveClusters(&active, reinterpret_cast<const void*>(fn), &cfg);
            if (*err != cudaSuccess) return -1;
            sn.occ_S = S;
            sn.occ_smem = smem;
            sn.occ_active = active;
        }
        if (active < 1) {
            *err = cudaErrorInvalidConfiguration;
            return -1;
        }
        n_clusters = active < n_clusters ? active : n_clusters;
    }
    // Two CTAs per SM (each takes 256 of the SM's 512 tensor-memory columns and under half its shared memory and
    // registers).  The occupancy calculator answers 1 for every kernel here that allocates tensor memory, whatever
    // its registers and shared memory, so it is not asked; measured at C = 256, batch 256 x 8 kv-heads: 0.076 ms per
    // step with one CTA of this form per SM, 0.059 ms with two, 0.065 ms with three (0.066 ms in the one-CTA form).
    if (small) n_clusters = 2 * c->sm_count;
    if (n_clusters > c->U) n_clusters = c->U;
    cfg.gridDim = dim3((unsigned)(n_clusters * S), 1, 1);
    *err = cudaLaunchKernelEx(&cfg, fn, *reinterpret_cast<const CUtensorMap*>(c->tmap_k),
                              *reinterpret_cast<const CUtensorMap*>(c->tmap_v),
                              *reinterpret_cast<const CUtensorMap*>(c->tmap_lo), a);
    if (*err != cudaSuccess) return -1;
    return 1;
}

}  // namespace bct
