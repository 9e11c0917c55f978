// Chunked stream / prefill kernel of the bounded-cache attention layer on the sm_100a tensor path.
//
// Algorithm 1 never assigns MK, so the write weights ww_t = softmax(wq_t . MK^T) of all tokens of
// a chunk are independent of one another ("Optimized for Parallelism": token-level parallel
// accumulation).  For a chunk of Tc tokens against a full cache this turns Tc decode steps into
// dense contractions over the resident tiles:
//     Sr = Q MK^T, Sw = Kc MK^T            scores of the chunk's read and write queries
//     Pr = softmax rows of Sr, WW = softmax rows of Sw
//     A  = Pr WW^T                          what token t's read sees of token s's write
//     O  = Pr MV + strict_tril(A) Vc        outputs: every token reads MV_{t-1}
//     MV += WW^T Vc                         Method step 4 for the Tc tokens at once
// While the cache still has Tc free slots the same kernel runs in fill mode: the chunk's keys and
// values are appended (TMA stores from the operand buffers), token t reads the resident slots plus
// the chunk's own slots s <= t (scores Q Kc^T, masked causally), and nothing is soft-written.
// One persistent CTA per (sequence, kv-head) unit and chunk at a time (C <= 16384 slots; see task_next for how the
// chunks are dealt round the CTAs); per chunk the cache
// streams through shared memory twice for MK (row statistics, then numerators) and once for MV
// (value and residual planes), instead of twice per token, and every product runs as tcgen05.mma
// with fp32 accumulators in tensor memory.  The write weights are always kept as bfloat16
// value + residual pairs (the state must not drift); with BCT_FLAG_PRECISE_READ the read uses MV's residual
// tile as well (one more product per tile), so that a long stream whose state grows large keeps the output
// precision.  (Measured over a 131072-token stream whose |MV| reaches 75: 0.040 max-abs with the value plane
// alone, 0.0075 with the residual tile, 0.0014 with residual numerators on top, which are therefore not kept.)
//   warp 16 producer : TMA loads (chunk operands, MK / MV tiles through a ring of stages)
//   warp 17 MMA      : issues all tensor-core work, commits to mbarriers
//   warps 0-15       : four threads per operand row (32 accumulator columns each): online row statistics, numerators, the write-back
//                      of MV rows, the intra-chunk term and the epilogue
// Every wait is bounded; a timeout sets the status word and the kernel runs to its end.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "bct_internal.h"
#include "bct_tc.cuh"

namespace bct {
namespace {

constexpr int kStRowWarps = 16;
constexpr int kStS = kStRowWarps * 32;   // row threads: four per operand row
constexpr int kStThreads = kStS + 64;    // + producer warp + MMA warp
constexpr int kStTile = 128;             // slots per tile
constexpr int kStHalf = 128 * 128;       // 64 columns (128 bytes) x 128 rows
constexpr int kStTileBytes = 2 * kStHalf;
constexpr int kStMaxStages = 4;
constexpr int kStMaxTc = 64;
constexpr int kStMaxCapacity = 16384;    // slots per unit: one CTA walks all tiles of a unit, twice per chunk
constexpr float kStNegBig = -3.0e38f;
// tensor-memory columns
constexpr int kColS0 = 0;     // score tile (pass 2, and buffer 0 of pass 1)
constexpr int kColO = 128;    // outputs  [row (t,g)] x [d]
constexpr int kColD = 256;    // MV increment of one tile [slot] x [d]; buffer 1 of the scores in pass 1
constexpr int kColA = 384;    // A = Pr WW^T  [row (t,g)] x [write token]

struct StArgs {
    char* out;
    unsigned long long* progress;  // [U]: (launch << 32 | chunks of this launch done) per unit, for the chunk-major schedule
    unsigned int launch;           // this launch's number
    int chunk_major;               // 1: the (unit, chunk) pairs are dealt round the CTAs chunk by chunk (see task_next)
    int* status;
    const float* eta;  // step size of each token's write, [B][T][Hkv], or NULL (all ones)
    int C, Hq, Hkv, U, T, t_begin, n_chunks, Tc;
    int fill, len0;  // fill = 1: the cache holds len0 slots and each chunk is appended (no soft write)
    int wtr, out_f32, precise;  // precise: the read uses MV's value + residual (one more product per tile)
    float read_scale, write_scale;
    float write_eps;  // write weights below it are dropped (0 with BCT_FLAG_DENSE_WRITE)
};

struct StSmem {
    int qall, vc, phi, plo, ring, bars, misc, total;
    int stages;    // ring stages of one tile each
    int plo_half;  // bytes between the two 64-column halves of the residual operand
};
// Shared-memory carve-up, the same on host and device.  Only the write rows keep a residual operand (at
// most 64 rows), which leaves room for four ring stages.  `wide`: chunks of more than 64 tokens (the
// write-only form, up to 128 write rows): a full residual buffer, twice the Vc and three stages.
__host__ __device__ inline StSmem st_smem(int wide) {
    StSmem L;
    L.stages = wide ? 3 : kStMaxStages;
    L.plo_half = wide ? kStHalf : kStMaxTc * 128;
    int off = 0;
    L.qall = off;
    off += kStTileBytes;        // [2 halves][128 rows][128 B]: G*Tc read queries, Tc write queries, zero rows
    L.vc = off;
    off += (wide ? 2 : 1) * kStMaxTc * 256;  // [2 halves][Tc rows][128 B]: the chunk's write key-value vectors
    L.phi = off;
    off += kStTileBytes;        // numerators / write weights of one tile, bfloat16 value
    L.plo = off;
    off += 2 * L.plo_half;      // ... and residual; reused for the row statistics and, after the last tile, the masked A operand
    L.ring = off;
    off += L.stages * kStTileBytes;
    L.bars = off;
    off += 32 * 8;
    L.misc = off;
    off += 64;                  // flags
    L.total = off + 1024;       // slack to align the base to 1024 bytes
    return L;
}

// use[s] of a stage picked at run time, without indexing the register array dynamically
__device__ __forceinline__ uint32_t& use_at(uint32_t (&u)[kStMaxStages], int s) {
    switch (s) {
        case 0: return u[0];
        case 1: return u[1];
        case 2: return u[2];
        default: return u[3];
    }
}

// 2^x (approximate, flushes denormals): every exponential of the kernel
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void st_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kStS) : "memory"); }

// value / residual split of 8 floats into two 16-byte chunks of bfloat16
__device__ __forceinline__ void split8(const float* e, uint4* hi, uint4* lo) {
    *hi = Chunk<__nv_bfloat16>::pack(e);
    float h[8], r[8];
    Chunk<__nv_bfloat16>::unpack(*hi, h);
#pragma unroll
    for (int i = 0; i < 8; ++i) r[i] = e[i] - h[i];
    *lo = Chunk<__nv_bfloat16>::pack(r);
}

template <int G>
__global__ void __launch_bounds__(kStThreads, 1)
stream_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmVhi,
                 const __grid_constant__ CUtensorMap tmVlo, const __grid_constant__ CUtensorMap tmQ,
                 const __grid_constant__ CUtensorMap tmKin, const __grid_constant__ CUtensorMap tmVin,
                 const __grid_constant__ CUtensorMap tmKapp, const __grid_constant__ CUtensorMap tmVapp,
                 const StArgs a) {
    extern __shared__ unsigned char st_smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(st_smem_raw) + 1023) & ~uintptr_t(1023));
    const StSmem L = st_smem(a.Tc > kStMaxTc);
    const int ns = L.stages;
    unsigned char* qall = smem + L.qall;
    unsigned char* vc = smem + L.vc;
    unsigned char* phi = smem + L.phi;
    unsigned char* plo = smem + L.plo;
    unsigned char* ring = smem + L.ring;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L.bars);
    uint64_t* full = bars;            // [4] tile landed (TMA transaction bytes)
    uint64_t* empty = bars + 20;      // [4] stage may be refilled (one arrival: MMA commit, or the producer after its store)
    uint64_t* qfull = bars + 6;       // the chunk's read and write queries landed
    uint64_t* vfull = bars + 5;       // the chunk's write key-value vectors landed
    uint64_t* qfree_q = bars + 4;     // every product that reads the query operand has been issued and is complete (commit)
    uint64_t* qfree = bars + 7;       // the chunk's outputs have been read from tensor memory (row-thread arrivals)
    uint64_t* sready = bars + 8;      // [2] score tile complete (commit)
    uint64_t* sfree = bars + 10;      // [2] score tile consumed (128 arrivals)
    uint64_t* pready = bars + 12;     // numerators of the tile written (128 arrivals)
    uint64_t* pfree = bars + 13;      // MMAs that read them complete (commit)
    uint64_t* dready = bars + 14;     // the tile's MV increment (and all earlier MMAs) complete (commit)
    uint64_t* dfree = bars + 15;      // increment consumed (128 arrivals)
    uint64_t* aready = bars + 16;     // masked A operand written (128 arrivals)
    uint64_t* oready = bars + 17;     // outputs complete (commit)
    uint64_t* ccready = bars + 19;    // fill mode: scores of the chunk's queries against its own keys (commit)
    uint64_t* wready = bars + 18;     // rewritten MV rows of the tile are in their ring stages (256 arrivals)
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L.misc);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L.misc + 8);
    float* rowstat = reinterpret_cast<float*>(plo);  // [4 quarters][128 rows](max, sum): between the two passes only

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const int Tc = a.Tc;
    const int nt_full = (a.C + kStTile - 1) / kStTile;
    // resident slots and tiles seen by chunk ch: everything once the cache is full, len0 + ch*Tc while it fills
    auto chunk_len = [&](int ch) { return a.fill ? a.len0 + ch * a.Tc : a.C; };
    auto chunk_tiles = [&](int ch) { return a.fill ? (a.len0 + ch * a.Tc + kStTile - 1) / kStTile : nt_full; };
    // The k-th (unit, chunk) pair of this CTA.  Unit-major: a CTA takes whole units, chunk after chunk.  Chunk-major:
    // pair i = chunk (i / U) of unit (i mod U) goes to CTA i mod gridDim, so that U units that do not divide by the
    // number of CTAs leave no CTA idle for a whole unit (256 units x 4 chunks on 148 CTAs: 7 turns instead of 8).  A
    // unit's chunks then run on different CTAs: chunk c waits until the unit's progress word says that chunk c - 1 of
    // this launch is in global memory (it was dealt a whole turn earlier, so the wait is over before it starts).
    // (Walked without divisions: the single-thread roles have nothing to hide them behind.  gridDim <= U.)
    auto task_first = [&](int& u, int& ch) {
        u = (int)blockIdx.x;
        ch = 0;
        return u < a.U;
    };
    auto task_next = [&](int& u, int& ch) {  // the pair after (u, ch) on this CTA; false when there is none
        if (a.chunk_major) {
            u += (int)gridDim.x;
            if (u >= a.U) {
                u -= a.U;
                ++ch;
            }
            return ch < a.n_chunks;
        }
        if (++ch < a.n_chunks) return true;
        ch = 0;
        u += (int)gridDim.x;
        return u < a.U;
    };
    const int n_read = Tc * G;         // rows [0, n_read): read queries (t, g); then Tc write rows
    const int Tcp = (Tc + 15) & ~15;   // the chunk padded to the 16-token step of the products (padding rows are zero)
    const int vc_half = Tcp * 128;     // bytes between the two 64-column halves of Vc
    // Ring use.  Pass 1 streams the MK tiles round the stages.  In pass 2 stage 0 takes the MK tiles, the
    // last stage the residual tiles of MV, and the stages between them the value tiles of MV: two of
    // them with four stages, so that tile t + 1's values arrive while tile t is rebuilt and stored.
    // use[s] counts the loads into stage s; every role walks the same sequence.
    const int st_vl = ns - 1;
    auto st_vh = [&](int t) { return ns == kStMaxStages ? 1 + (t & 1) : 1; };
    const bool load_vl = !a.fill || a.precise;  // the residual tiles feed the write-back and the precise read only
    auto pass1_advance = [&](uint32_t (&use)[kStMaxStages], int nt) {
#pragma unroll
        for (int st = 0; st < kStMaxStages; ++st)
            if (st < ns && nt > st) use[st] += (uint32_t)((nt - st + ns - 1) / ns);
    };
    auto pass2_advance = [&](uint32_t (&use)[kStMaxStages], int nt) {
        use[0] += nt;
        if (ns == kStMaxStages) {
            use[1] += (nt + 1) >> 1;
            use[2] += nt >> 1;
        } else {
            use[1] += nt;
        }
        if (load_vl) use_at(use, st_vl) += nt;
    };
    auto vh_use = [&](uint32_t (&use)[kStMaxStages], int t) {
        return ns == kStMaxStages ? ((t & 1) ? use[2] : use[1]) + (uint32_t)(t >> 1) : use[1] + (uint32_t)t;
    };

    if (tid == 0) {
        for (int i = 0; i < kStMaxStages; ++i) {
            mbar_init(&full[i], 1);
            mbar_init(&empty[i], 1);
        }
        mbar_init(qfull, 1);
        mbar_init(vfull, 1);
        mbar_init(qfree_q, 1);
        mbar_init(qfree, kStS);
        mbar_init(&sready[0], 1);
        mbar_init(&sready[1], 1);
        mbar_init(&sfree[0], kStS);
        mbar_init(&sfree[1], kStS);
        mbar_init(pready, kStS);
        mbar_init(pfree, 1);
        mbar_init(dready, 1);
        mbar_init(dfree, kStS);
        mbar_init(aready, kStS);
        mbar_init(oready, 1);
        mbar_init(wready, kStS);
        mbar_init(ccready, 1);
        *abort_flag = 0;
        fence_mbar_init_cluster();
    }
    // rows of the query operand beyond the chunk's G*Tc + Tc, and rows of Vc beyond Tc, stay zero for good
    for (int i = tid; i < (L.phi - L.vc) / 16; i += kStThreads) reinterpret_cast<uint4*>(vc)[i] = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < kStTileBytes / 16; i += kStThreads) reinterpret_cast<uint4*>(qall)[i] = make_uint4(0, 0, 0, 0);
    if (warp == kStRowWarps + 1) tmem_alloc(tmem_slot, 512);
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

#define ST_WAIT(bar, parity, site)                                              \
    if (!mbar_wait_abortable(bar, (parity) & 1, abort_flag)) {      \
        report_timeout(a.status, site);                                         \
        *abort_flag = 1;                                                        \
    }

    if (warp == kStRowWarps) {
        // =========================== producer ===========================
        if (lane == 0) {
            uint32_t qn = 0, nw = 0;
            int pre = 0;  // tiles of the next pair's pass 1 that have been asked for already
            int handed_u = -1, handed_ch = 0;  // a finished chunk whose progress word has not been written yet
            // The pair before is complete in global memory (its stores were waited for): say so in its unit's progress
            // word.  The release takes about half a microsecond and only a CTA a whole turn behind waits for it, so it
            // is written after the next pair's first copies have been asked for, and in any case before this CTA waits
            // for anything another CTA has to hand over.
            auto hand_over = [&]() {
                if (handed_u < 0) return;
                fence_proxy_async_global();
                const unsigned long long done = ((unsigned long long)a.launch << 32) | (unsigned int)handed_ch;
                asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(a.progress + handed_u), "l"(done) : "memory");
                handed_u = -1;
            };
            unsigned long long rows_stored = 0;  // MV rows this CTA has stored back
            uint32_t use[kStMaxStages] = {0, 0, 0, 0};
            auto load_tile = [&](const CUtensorMap* map, int u, int t, int stage) {
                const uint32_t n = use_at(use, stage)++;
                if (n > 0) ST_WAIT(&empty[stage], n - 1, 31);
                unsigned char* dst = ring + (size_t)stage * kStTileBytes;
                mbar_arrive_expect_tx(&full[stage], kStTileBytes);
                tma_load_3d(dst, map, 0, t * kStTile, u, &full[stage]);
                tma_load_3d(dst + kStHalf, map, 64, t * kStTile, u, &full[stage]);
            };
            // A cache of a single tile (C <= 128 slots) stays resident in shared memory for all chunks of the launch:
            // MK keeps stage 0, MV's value and residual tiles keep their stages, where the row threads rebuild them
            // chunk after chunk.  The loads after the first chunk and the stores before the last one are left out;
            // the barriers are handed over as if they had happened, so the other roles do not change.
            const bool resident = !a.fill && nt_full == 1 && a.n_chunks > 1 && !a.chunk_major;
            auto keep_tile = [&](int stage) {   // the stage already holds the tile: complete the barrier's phase without a copy
                const uint32_t n = use_at(use, stage)++;
                if (n > 0) ST_WAIT(&empty[stage], n - 1, 37);
                mbar_arrive(&full[stage]);
            };
            // read and write queries of chunk ch of unit u into the query operand
            auto load_queries = [&](int u, int ch) {
                const int b = u / a.Hkv, h = u - b * a.Hkv;
                const int t0 = a.t_begin + ch * Tc;
                mbar_arrive_expect_tx(qfull, (uint32_t)(Tc * (G + 1) * 256));
                if (G > 0) {
                    tma_load_4d(qall, &tmQ, 0, h * G, t0, b, qfull);
                    tma_load_4d(qall + kStHalf, &tmQ, 64, h * G, t0, b, qfull);
                }
                tma_load_4d(qall + n_read * 128, &tmKin, 0, h, t0, b, qfull);
                tma_load_4d(qall + kStHalf + n_read * 128, &tmKin, 64, h, t0, b, qfull);
            };
            // The query operand is free once the last scores of a chunk are complete, well before the
            // chunk's last tile is stored: the next chunk's queries are asked for at that point.
            auto next_queries = [&](int u, int ch) {
                int u2 = u, ch2 = ch;
                if (!task_next(u2, ch2)) return;
                ST_WAIT(qfree_q, qn, 32);
                if (a.fill) bulk_wait_read();  // the appended keys have been read out of the operand
                load_queries(u2, ch2);
            };
            for (int u = 0, ch = 0, more = task_first(u, ch); more; more = task_next(u, ch), ++qn) {
                const int b = u / a.Hkv, h = u - b * a.Hkv;
                {
                    const int t0 = a.t_begin + ch * Tc;
                    const int nt = chunk_tiles(ch);
                    // The unit's previous chunk ran on another CTA: its rows (and appended keys) must be in global memory
                    // before this chunk's copies read them.  While the cache fills that is every tile copy; with a full
                    // cache MK is constant and only the MV tiles of pass 2 depend on it, so the check comes after pass 1's
                    // copies have been issued, off the start of the pair.
                    auto wait_for_previous_chunk = [&]() {
                        if (!a.chunk_major || ch == 0) return;
                        const unsigned long long want = ((unsigned long long)a.launch << 32) | (unsigned int)ch;
                        bool seen = false;
                        for (uint32_t i = 0; i < (*abort_flag ? 1024u : kWaitLimit) && !seen; ++i) {
                            unsigned long long got;
                            asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(got) : "l"(a.progress + u) : "memory");
                            seen = got == want;
                            if (!seen && i > 64) __nanosleep(i > 4096 ? 256 : 32);
                        }
                        if (!seen) {
                            report_timeout(a.status, 30);
                            *abort_flag = 1;
                        }
                        fence_proxy_async_global();
                    };
                    if (a.fill) {
                        hand_over();
                        wait_for_previous_chunk();
                    }
                    // the first MK tiles of pass 1 do not depend on the chunk's operands: ask for them first
                    const int n_early = nt < ns - 1 ? nt : ns - 1;
                    int st1 = pre;  // pass-1 stage of the next tile, t mod ns without the division
                    for (int t = pre; t < n_early; ++t) {  // (the first `pre` tiles were asked for during the pair before)
                        if (resident && ch > 0)
                            keep_tile(st1);
                        else
                            load_tile(&tmK, u, t, st1);
                        if (++st1 == ns) st1 = 0;
                    }
                    pre = 0;
                    if (qn == 0) load_queries(u, ch);
                    if (qn > 0) ST_WAIT(oready, qn - 1, 35);  // the previous chunk's last product has read Vc
                    mbar_arrive_expect_tx(vfull, (uint32_t)(Tc * 256));
                    tma_load_4d(vc, &tmVin, 0, h, t0, b, vfull);
                    tma_load_4d(vc + vc_half, &tmVin, 64, h, t0, b, vfull);
                    if (a.fill) {
                        // fill phase: the chunk's keys and values are appended at slots len .. len + Tc - 1
                        // straight from the operand buffers (the residual plane is zero there already)
                        ST_WAIT(qfull, qn, 34);
                        ST_WAIT(vfull, qn, 36);
                        const int len = chunk_len(ch);
                        tma_store_3d(&tmKapp, 0, len, u, qall + n_read * 128);
                        tma_store_3d(&tmKapp, 64, len, u, qall + kStHalf + n_read * 128);
                        tma_store_3d(&tmVapp, 0, len, u, vc);
                        tma_store_3d(&tmVapp, 64, len, u, vc + vc_half);
                        bulk_commit();
                    }
                    for (int t = n_early; t < nt; ++t) {  // pass 1: row statistics
                        load_tile(&tmK, u, t, st1);
                        if (++st1 == ns) st1 = 0;
                    }
                    // pass 2: numerators, outputs, update.  The row threads put the rewritten MV rows back
                    // into the two ring stages the tile came in; they go home as TMA stores from here.
                    // The MK tile is asked for two tiles ahead (its stage is free as soon as the scores of the
                    // tile before it are issued, long before tile t is stored), the values one tile ahead when
                    // there are two value stages.  The residual stage is stored and refilled first: the next
                    // tile's write-back waits for it.
                    const bool two_vh = ns == kStMaxStages;
                    if (!a.fill) {
                        hand_over();
                        wait_for_previous_chunk();
                    }
                    if (nt > 0 && resident) {
                        keep_tile(0);  // pass 1 left the MK tile in stage 0
                        if (ch == 0) {
                            load_tile(&tmVhi, u, 0, st_vh(0));
                            load_tile(&tmVlo, u, 0, st_vl);
                        } else {
                            keep_tile(st_vh(0));
                            keep_tile(st_vl);
                        }
                    } else if (nt > 0) {
                        load_tile(&tmK, u, 0, 0);
                        load_tile(&tmVhi, u, 0, st_vh(0));
                        if (load_vl) load_tile(&tmVlo, u, 0, st_vl);
                        if (nt > 1) load_tile(&tmK, u, 1, 0);
                        if (nt > 1 && two_vh) load_tile(&tmVhi, u, 1, st_vh(1));
                    }
                    if (nt == 0) next_queries(u, ch);
                    for (int t = 0; t < nt; ++t) {
                        if (t + 2 < nt) load_tile(&tmK, u, t + 2, 0);
                        if (t == nt - 1) {
                            next_queries(u, ch);
                            // With a full cache MK never changes, so the first tiles of the next pair's pass 1 depend on
                            // nothing that is still in flight: they are asked for now, into the stages that are already
                            // free (the MK stage after the last scores; stage 1 when the tile before the last one had its
                            // values there), instead of after this pair's last stores.  Without this the tensor pipe and the
                            // row threads wait 4-5 us for MK tiles at the start of every pair.
                            int u2 = u, ch2 = ch;
                            if (!a.fill && !resident && task_next(u2, ch2)) {
                                load_tile(&tmK, u2, 0, 0);
                                pre = 1;
                                if (nt >= 2 && ns > 2 && st_vh(nt - 2) == 1 && st_vh(nt - 1) != 1) {
                                    load_tile(&tmK, u2, 1, 1);
                                    pre = 2;
                                }
                            }
                        }
                        const int pvh = st_vh(t);
                        if (resident && ch + 1 < a.n_chunks) {
                            // the rebuilt tile is the next chunk's MV: nothing goes to HBM yet
                            ST_WAIT(wready, nw, 33);
                            ++nw;
                            mbar_arrive(&empty[st_vl]);
                            mbar_arrive(&empty[pvh]);
                            continue;
                        }
                        if (!a.fill) {
                            ST_WAIT(wready, nw, 33);
                            ++nw;
                            unsigned char* sh = ring + (size_t)pvh * kStTileBytes;
                            unsigned char* sl = ring + (size_t)st_vl * kStTileBytes;
                            tma_store_3d(&tmVlo, 0, t * kStTile, u, sl);
                            if (two_vh) bulk_commit();  // (the two halves as groups of their own)
                            tma_store_3d(&tmVlo, 64, t * kStTile, u, sl + kStHalf);
                            bulk_commit();
                            if (two_vh) {
                                // The residual stage first and alone: the next tile's rebuild waits for its refill, while
                                // the next value tile is in its other stage already (0.381 -> 0.370 ms per 256-token step).
                                // Each half is refilled as soon as it has been read out.
                                bulk_wait_read_but_one();
                                if (t + 1 < nt) {
                                    mbar_arrive_expect_tx(&full[st_vl], kStTileBytes);
                                    tma_load_3d(sl, &tmVlo, 0, (t + 1) * kStTile, u, &full[st_vl]);
                                }
                                bulk_wait_read();
                                mbar_arrive(&empty[st_vl]);
                                if (t + 1 < nt) {
                                    const uint32_t n = use_at(use, st_vl)++;
                                    ST_WAIT(&empty[st_vl], n - 1, 31);  // (this thread's own arrival, kept for the count)
                                    tma_load_3d(sl + kStHalf, &tmVlo, 64, (t + 1) * kStTile, u, &full[st_vl]);
                                }
                                tma_store_3d(&tmVhi, 0, t * kStTile, u, sh);
                                tma_store_3d(&tmVhi, 64, t * kStTile, u, sh + kStHalf);
                                bulk_commit();
                            } else {  // one value stage: the next tile waits for both refills
                                tma_store_3d(&tmVhi, 0, t * kStTile, u, sh);
                                tma_store_3d(&tmVhi, 64, t * kStTile, u, sh + kStHalf);
                                bulk_commit();
                                bulk_wait_read_but_one();
                                mbar_arrive(&empty[st_vl]);
                                if (t + 1 < nt) load_tile(&tmVlo, u, t + 1, st_vl);
                            }
                        } else if (t + 1 < nt && load_vl) {
                            load_tile(&tmVlo, u, t + 1, st_vl);
                        }
                        if (t + 2 < nt && load_vl) {  // and the one after it towards L2: its load must not wait for HBM
                            tma_prefetch_3d(&tmVlo, 0, (t + 2) * kStTile, u);
                            tma_prefetch_3d(&tmVlo, 64, (t + 2) * kStTile, u);
                            if (!two_vh) {  // one value stage: the same for the values
                                tma_prefetch_3d(&tmVhi, 0, (t + 2) * kStTile, u);
                                tma_prefetch_3d(&tmVhi, 64, (t + 2) * kStTile, u);
                            }
                        }
                        if (!a.fill) {
                            bulk_wait_read();
                            mbar_arrive(&empty[pvh]);
                        }
                        if (two_vh) {
                            if (t + 2 < nt) load_tile(&tmVhi, u, t + 2, st_vh(t + 2));
                        } else if (t + 1 < nt) {
                            load_tile(&tmVhi, u, t + 1, st_vh(t + 1));
                        }
                    }
                    bulk_wait_all();  // the next chunk reads these rows again
                    if (a.chunk_major && ch + 1 < a.n_chunks) {
                        // ... on another CTA: the unit is handed over (hand_over) once the next pair's first copies are out
                        handed_u = u;
                        handed_ch = ch + 1;
                    }
                    // every tile of the unit was rebuilt and stored (a resident tile goes home after the last chunk only)
                    if (!a.fill && (!resident || ch + 1 == a.n_chunks)) rows_stored += (unsigned long long)a.C;
                }
            }
            hand_over();
            if (rows_stored > 0) atomicAdd(reinterpret_cast<unsigned long long*>(a.status + kStatusRowsWord), rows_stored);
        }
        __syncwarp();
    } else if (warp == kStRowWarps + 1) {
        // =========================== MMA issuer ===========================
        if (lane == 0) {
            constexpr uint32_t id_scores = instr_desc_mn(128, 128, false, false);  // Qall (K) x tile (K)
            constexpr uint32_t id_out = instr_desc_mn(128, 128, false, true);      // P (K) x V tile (MN)
            constexpr uint32_t id_delta = instr_desc_mn(128, 128, true, true);     // WW^T (MN) x Vc (MN)
            const uint32_t id_a = instr_desc_mn(128, (uint32_t)(Tcp > kStMaxTc ? kStMaxTc : Tcp), false, false);  // P (K) x WW (K)
            uint32_t qn = 0, su0 = 0, su1 = 0, np = 0, nd = 0;
            uint32_t use[kStMaxStages] = {0, 0, 0, 0};
            const uint32_t plo_row0 = (uint32_t)n_read;  // first operand row the residual buffer holds
            // descriptors at shared address 0 (K-major; MN-major with the half strides of the tiles, of Vc and of
            // the residual operand): the address field is added per use, addresses stay below 256 KiB
            const DescKind dk(smem_desc(0, 16, 1024)), dmn(smem_desc(0, kStHalf, 1024));
            const DescKind dvc(smem_desc(0, (uint32_t)vc_half, 1024)), dpl(smem_desc(0, (uint32_t)L.plo_half, 1024));
            // the operand buffers in the 16-byte units of the address field
            const uint32_t q16 = desc_addr16(smem_u32(qall)), vc16 = desc_addr16(smem_u32(vc)), phi16 = desc_addr16(smem_u32(phi));
            const uint32_t plo16 = desc_addr16(smem_u32(plo)), ring16 = desc_addr16(smem_u32(ring));
            const uint32_t qw16 = q16 + n_read * 8, pw16 = phi16 + n_read * 8;  // the write rows of the two operand buffers
            const uint32_t plw16 = plo16 + ((uint32_t)n_read - plo_row0) * 8;
            auto scores = [&](uint32_t col, int stage) {
                const uint32_t t16 = ring16 + stage * (kStTileBytes / 16);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t o = ((kk >> 2) * kStHalf + (kk & 3) * 32) / 16;
                    umma_bf16(tmem_base + col, dk.at(q16 + o), dk.at(t16 + o), id_scores, kk > 0);
                }
            };
            for (int u = 0, ch = 0, more = task_first(u, ch); more; more = task_next(u, ch), ++qn) {
                {
                    ST_WAIT(qfull, qn, 41);
                    tc_fence_after();
                    const int nt = chunk_tiles(ch);
                    if (a.fill) {
                        // scores of the chunk's queries against the chunk's own keys (rows n_read.. of the
                        // operand buffer), into the columns the full phase uses for A
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {
                            const uint32_t o = ((kk >> 2) * kStHalf + (kk & 3) * 32) / 16;
                            umma_bf16(tmem_base + kColA, dk.at(q16 + o), dk.at(qw16 + o), id_a, kk > 0);
                        }
                        umma_commit(ccready);
                        if (nt == 0) umma_commit(qfree_q);  // nothing else reads the query operand
                    }
                    for (int t = 0, st1 = 0; t < nt; ++t, st1 = (st1 + 1 == ns ? 0 : st1 + 1)) {  // pass 1
                        const int stage = st1;
                        const int buf = t & 1;
                        ST_WAIT(&full[stage], use_at(use, stage), 42);
                        ++use_at(use, stage);
                        uint32_t& su = buf ? su1 : su0;
                        if (su > 0) ST_WAIT(&sfree[buf], su - 1, 43);
                        if (buf == 1 && nd > 0) ST_WAIT(dfree, nd - 1, 51);  // buffer 1 is the increment's columns
                        tc_fence_after();
                        scores(buf ? kColD : kColS0, stage);
                        umma_commit(&sready[buf]);
                        umma_commit(&empty[stage]);
                        ++su;
                    }
                    // pass 2: the scores of tile t + 1 are issued before the products of tile t, so that the row
                    // threads turn them into numerators while the tensor pipe works on tile t
                    auto issue_scores = [&](int t) {
                        ST_WAIT(&full[0], use[0] + (uint32_t)t, 44);
                        if (su0 > 0) ST_WAIT(&sfree[0], su0 - 1, 45);
                        tc_fence_after();
                        scores(kColS0, 0);
                        umma_commit(&sready[0]);
                        umma_commit(&empty[0]);
                        if (t == nt - 1) umma_commit(qfree_q);  // the last product that reads the query operand
                        ++su0;
                    };
                    // the previous chunk's outputs have left tensor memory; this chunk's Vc has landed
                    if (qn > 0) ST_WAIT(qfree, qn - 1, 52);
                    ST_WAIT(vfull, qn, 53);
                    tc_fence_after();
                    if (nt > 0) issue_scores(0);
                    for (int t = 0; t < nt; ++t) {
                        if (t + 1 < nt) issue_scores(t + 1);
                        const int vh = st_vh(t), vl = st_vl;
                        ST_WAIT(pready, np, 46);
                        ++np;
                        ST_WAIT(&full[vh], vh_use(use, t), 47);
                        tc_fence_after();
                        const uint32_t vh16 = ring16 + vh * (kStTileBytes / 16), vl16 = ring16 + vl * (kStTileBytes / 16);
                        // outputs: P x MV_value, accumulated over the tiles (none in the write-only form, G = 0).  Issued
                        // first: they need nothing the rebuild of the previous tile's rows still holds.
#pragma unroll
                        for (int kk = 0; kk < (G > 0 ? 8 : 0); ++kk) {
                            const uint32_t po = ((kk >> 2) * kStHalf + (kk & 3) * 32) / 16;
                            umma_bf16(tmem_base + kColO, dk.at(phi16 + po), dmn.at(vh16 + kk * 128), id_out, (t > 0) || (kk > 0));
                        }
                        // ... + P x MV_residual with PRECISE_READ: the residual tile arrives once the previous tile's
                        // rows have been stored out of its stage
                        auto residual_outputs = [&]() {
                            ST_WAIT(&full[vl], use_at(use, vl) + (uint32_t)t, 48);
                            tc_fence_after();
#pragma unroll
                            for (int kk = 0; kk < (G > 0 ? 8 : 0); ++kk) {
                                const uint32_t po = ((kk >> 2) * kStHalf + (kk & 3) * 32) / 16;
                                umma_bf16(tmem_base + kColO, dk.at(phi16 + po), dmn.at(vl16 + kk * 128), id_out, true);
                            }
                        };
                        if (a.fill) {
                            // no soft write while the cache fills: the stages are free once the outputs are done
                            if (a.precise) residual_outputs();
                            umma_commit(pfree);
                            umma_commit(&empty[vh]);
                            if (load_vl) umma_commit(&empty[vl]);
                            continue;
                        }
                        if (nd > 0) ST_WAIT(dfree, nd - 1, 49);  // the previous tile's increment has been read
                        tc_fence_after();
                        // increment of this tile's MV rows: (WW + WW_residual)^T x Vc, 16 tokens per step
                        for (int kk = 0; kk < Tcp / 16; ++kk) {
                            const uint64_t vd = dvc.at(vc16 + kk * 128);
                            umma_bf16(tmem_base + kColD, dmn.at(pw16 + kk * 128), vd, id_delta, kk > 0);
                            umma_bf16(tmem_base + kColD, dpl.at(plw16 + kk * 128), vd, id_delta, true);
                        }
                        if (a.precise) residual_outputs();
                        umma_commit(dready);  // the write-back may start: outputs and increment are complete
                        // A += P x WW^T over this tile's slots (write rows start at n_read)
#pragma unroll
                        for (int kk = 0; kk < (G > 0 ? 8 : 0); ++kk) {
                            const uint32_t po = ((kk >> 2) * kStHalf + (kk & 3) * 32) / 16;
                            umma_bf16(tmem_base + kColA, dk.at(phi16 + po), dk.at(pw16 + po), id_a, (t > 0) || (kk > 0));
                        }
                        umma_commit(pfree);
                        ++nd;
                    }
                    pass2_advance(use, nt);
                    // intra-chunk term: O += strict_tril(A) x Vc (fill phase: the causal numerators of the
                    // chunk's own slots, value + residual, times Vc)
                    ST_WAIT(aready, qn, 50);
                    tc_fence_after();
                    for (int kk = 0; kk < (G > 0 ? Tcp / 16 : 0); ++kk) {
                        umma_bf16(tmem_base + kColO, dk.at(plo16 + kk * 2), dvc.at(vc16 + kk * 128), id_out, (nt > 0) || (kk > 0));
                    }
                    umma_commit(oready);
                }
            }
        }
        __syncwarp();
    } else {
        // =========================== row threads: statistics, numerators, write-back, epilogue ===========================
        // Four threads per operand row (tensor-memory lane): thread quarter cq works on columns
        // [32 cq, 32 cq + 32) of every 128-column accumulator.  Exponentials are taken in base 2:
        // scores are multiplied by scale * log2(e) once, maxima are kept in that domain.
        const int r = tid & 127;
        const int cq = tid >> 7;
        const uint32_t lane_base = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + cq * 32;
        const bool is_read = r < n_read;
        const bool is_write = !is_read && r < n_read + Tc;
        const int my_t = is_read ? r / (G > 0 ? G : 1) : (is_write ? r - n_read : 0);  // token of the chunk this row belongs to
        const int my_g = is_read ? r - my_t * G : 0;
        const float c2 = (is_read ? a.read_scale : a.write_scale) * 1.4426950408889634f;
        const int sw = r & 7;                                // swizzle phase of this row
        const int poff = (cq >> 1) * kStHalf + r * 128;      // this thread's 64 bytes: chunks (cq & 1) * 4 + j
        const int pch = (cq & 1) * 4;
        const bool active = is_read || (is_write && !a.fill);  // rows that produce numerators
        // rows whose residual the increment's product reads: the write rows and the zero rows that pad the chunk to 16 tokens
        const bool lo_row = !is_read && r < n_read + Tcp;
        uint32_t qn = 0, su0 = 0, su1 = 0, np = 0, nd = 0;
        uint32_t use[kStMaxStages] = {0, 0, 0, 0};
        const int lo_off = (cq >> 1) * L.plo_half + (r - n_read) * 128;  // the residual buffer holds the write rows only
        for (int u = 0, ch = 0, more = task_first(u, ch); more; more = task_next(u, ch), ++qn) {
            const int b = u / a.Hkv, h = u - b * a.Hkv;
            {
                const int t0 = a.t_begin + ch * Tc;
                const int nt = chunk_tiles(ch);
                const int clen = chunk_len(ch);
                // ---- pass 1: online maximum and sum of this quarter row's scaled scores over the resident slots ----
                float m = kStNegBig, l = 0.f;
                for (int t = 0; t < nt; ++t) {
                    const int buf = t & 1;
                    uint32_t& su = buf ? su1 : su0;
                    ST_WAIT(&sready[buf], su, 61);
                    ++su;
                    tc_fence_after();
                    const int n_valid = min(kStTile, clen - t * kStTile) - cq * 32;
                    float x[32];
                    tmem_ld32(lane_base + (buf ? kColD : kColS0), x);
                    tc_fence_before();
                    mbar_arrive(&sfree[buf]);  // the scores are in registers
                    if (n_valid >= 32) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) x[i] *= c2;
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) x[i] = (i < n_valid) ? x[i] * c2 : kStNegBig;
                    }
                    float b0 = fmaxf(x[0], x[1]), b1 = fmaxf(x[2], x[3]), b2 = fmaxf(x[4], x[5]), b3 = fmaxf(x[6], x[7]);
#pragma unroll
                    for (int i = 8; i < 32; i += 8) {
                        b0 = fmaxf(b0, fmaxf(x[i], x[i + 1]));
                        b1 = fmaxf(b1, fmaxf(x[i + 2], x[i + 3]));
                        b2 = fmaxf(b2, fmaxf(x[i + 4], x[i + 5]));
                        b3 = fmaxf(b3, fmaxf(x[i + 6], x[i + 7]));
                    }
                    const float mn = fmaxf(m, fmaxf(fmaxf(b0, b1), fmaxf(b2, b3)));
                    if (!is_write) {  // read rows need only the maximum here: their sum is taken from the numerators of pass 2
                        m = mn;
                        continue;
                    }
                    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        s0 += ex2(x[i] - mn);
                        s1 += ex2(x[i + 1] - mn);
                        s2 += ex2(x[i + 2] - mn);
                        s3 += ex2(x[i + 3] - mn);
                    }
                    l = l * ex2(m - mn) + ((s0 + s1) + (s2 + s3));
                    m = mn;
                }
                if (a.fill) {
                    // fill phase: token t also sees the chunk's own slots s <= t (it is appended before it reads);
                    // thread quarter cq covers chunk tokens [16 cq, 16 cq + 16)
                    ST_WAIT(ccready, qn, 68);
                    tc_fence_after();
                    float cc[16];
                    const uint32_t cbase = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + kColA + cq * 16;
                    tmem_ld16(cbase, cc);
                    float bm = kStNegBig;
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int s = cq * 16 + i;
                        cc[i] = (is_read && s < Tc && s <= my_t) ? cc[i] * c2 : kStNegBig;
                        bm = fmaxf(bm, cc[i]);
                    }
                    m = fmaxf(m, bm);  // read rows only (write rows see nothing here): the sum comes with the numerators
                }
                // combine the four quarters of the row
                rowstat[(cq * 128 + r) * 2] = m;
                rowstat[(cq * 128 + r) * 2 + 1] = l;
                st_sync();
                {
                    float mn = m;
#pragma unroll
                    for (int o = 1; o < 4; ++o) mn = fmaxf(mn, rowstat[(((cq + o) & 3) * 128 + r) * 2]);
                    l *= ex2(m - mn);
#pragma unroll
                    for (int o = 1; o < 4; ++o) {
                        const int idx = (((cq + o) & 3) * 128 + r) * 2;
                        l += rowstat[idx + 1] * ex2(rowstat[idx] - mn);
                    }
                    m = mn;
                }
                st_sync();  // the statistics have been read: the buffer goes back to the residual operand
                pass1_advance(use, nt);
                float lr = 0.f;  // read rows: sum of this thread's numerators
                // write weights are stored normalised and carry the token's step size:
                // MV += sum_t eta_t ww_t^T wv_t, and A = Pr WW^T then holds eta_t as well
                float winv = 1.f, weta = 1.f;
                if (is_write && !a.fill) {
                    winv = 1.f / l;
                    // (a ragged last chunk of the write-only form has rows past the last token: their Vc rows are zero)
                    if (a.eta != nullptr && !a.fill && t0 + my_t < a.T) weta = a.eta[((size_t)b * a.T + t0 + my_t) * a.Hkv + h];
                }

                // ---- pass 2: numerators of each tile, then the write-back of its MV rows.  The numerators of
                // ---- tile t + 1 are taken (into registers) while the tensor pipe works on tile t ----
                float e[32];
                auto numerators = [&](int t) {
                    ST_WAIT(&sready[0], su0, 62);
                    ++su0;
                    tc_fence_after();
                    const int n_valid = min(kStTile, clen - t * kStTile) - cq * 32;
                    tmem_ld32(lane_base + kColS0, e);
                    tc_fence_before();
                    mbar_arrive(&sfree[0]);  // the scores are in registers: the next tile's may be computed
                    if (!active) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) e[i] = 0.f;
                    } else if (n_valid >= 32) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) e[i] = ex2(fmaf(e[i], c2, -m));
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) e[i] = (i < n_valid) ? ex2(fmaf(e[i], c2, -m)) : 0.f;
                    }
                    if (is_write) {
                        // ww_j below write_eps: the slot keeps its row (and a read that follows the write sees none of it)
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const float ww = e[i] * winv;
                            e[i] = ww >= a.write_eps ? ww * weta : 0.f;
                        }
                    } else {
                        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
                        for (int i = 0; i < 32; i += 4) {
                            s0 += e[i];
                            s1 += e[i + 1];
                            s2 += e[i + 2];
                            s3 += e[i + 3];
                        }
                        lr += (s0 + s1) + (s2 + s3);
                    }
                };
                // the numerators / write weights held in e, into the operand buffers, once the products that read the
                // previous ones are complete
                auto store_operand = [&]() {
                    if (np > 0) ST_WAIT(pfree, np - 1, 63);
                    if (lo_row) {  // write weights always keep the residual
#pragma unroll
                        for (int j = 0; j < 4; ++j) {  // 16-byte chunk = 8 slots
                            uint4 hi, lo;
                            split8(e + 8 * j, &hi, &lo);
                            const int off = poff + (((pch + j) ^ sw) * 16);
                            *reinterpret_cast<uint4*>(phi + off) = hi;
                            *reinterpret_cast<uint4*>(plo + lo_off + (((pch + j) ^ sw) * 16)) = lo;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            *reinterpret_cast<uint4*>(phi + poff + (((pch + j) ^ sw) * 16)) =
                                Chunk<__nv_bfloat16>::pack(e + 8 * j);
                    }
                    fence_proxy_async_smem();
                    mbar_arrive(pready);
                    ++np;
                };
                // Order of a tile's turn: its operand goes out as soon as the products of the tile before it are complete,
                // then the numerators of the next tile are taken into registers (the tensor pipe works on this tile
                // meanwhile), then this tile's rows are rebuilt.  (Measured against the two other orders, operand of
                // tile t + 1 before or after the rebuild of tile t: 0.381 ms against 0.414 and 0.396 per 256-token step.)
                if (nt > 0) numerators(0);
                for (int t = 0; t < nt; ++t) {
                    store_operand();
                    if (t + 1 < nt) numerators(t + 1);
                    if (a.fill) continue;  // no soft write while the cache fills: operands only

                    // the tile's MV rows: value + residual + increment, split again, stored (this thread: 32 of the 128 d)
                    const int vh = st_vh(t), vl = st_vl;
                    ST_WAIT(&full[vh], vh_use(use, t), 64);
                    ST_WAIT(&full[vl], use_at(use, vl) + (uint32_t)t, 65);
                    ST_WAIT(dready, nd, 66);
                    ++nd;
                    tc_fence_after();
                    {
                        unsigned char* th = ring + (size_t)vh * kStTileBytes + poff;
                        unsigned char* tl = ring + (size_t)vl * kStTileBytes + poff;
                        // rows past C of a ragged last tile are clipped by the store
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {  // 16 columns at a time
                            float dx[16];
                            tmem_ld16(lane_base + kColD + hh * 16, dx);
                            if (hh == 1) {
                                tc_fence_before();
                                mbar_arrive(dfree);
                            }
#pragma unroll
                            for (int jj = 0; jj < 2; ++jj) {
                                const int off = ((pch + hh * 2 + jj) ^ sw) * 16;
                                float vh8[8], vl8[8], nv[8];
                                Chunk<__nv_bfloat16>::unpack(*reinterpret_cast<const uint4*>(th + off), vh8);
                                Chunk<__nv_bfloat16>::unpack(*reinterpret_cast<const uint4*>(tl + off), vl8);
#pragma unroll
                                for (int q8 = 0; q8 < 8; ++q8) nv[q8] = (vh8[q8] + vl8[q8]) + dx[8 * jj + q8];
                                uint4 hi, lo;
                                split8(nv, &hi, &lo);
                                *reinterpret_cast<uint4*>(th + off) = hi;  // in place: the producer stores the stage
                                *reinterpret_cast<uint4*>(tl + off) = lo;
                            }
                        }
                    }
                    fence_proxy_async_smem();
                    mbar_arrive(wready);
                }
                pass2_advance(use, nt);

                // ---- intra-chunk term: thread quarter cq covers chunk tokens [16 cq, 16 cq + 16) ----
                if (a.fill) {
                    // fill phase: numerators of the chunk's own slots, 2^(score - m) for s <= t, as value + residual
                    if (np > 0) ST_WAIT(pfree, np - 1, 69);  // the last tile's MMAs have read the residual buffer
                    tc_fence_after();
                    if (cq * 16 < Tc) {
                        float cc[16];
                        const uint32_t cbase = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + kColA + cq * 16;
                        tmem_ld16(cbase, cc);
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            const int c = cq * 2 + j;
                            float z[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                const int s = c * 8 + e;
                                z[e] = (is_read && s <= my_t) ? ex2(fmaf(cc[8 * j + e], c2, -m)) : 0.f;
                                lr += z[e];
                            }
                            *reinterpret_cast<uint4*>(plo + r * 128 + ((c ^ sw) * 16)) = Chunk<__nv_bfloat16>::pack(z);
                        }
                    }
                    tc_fence_before();
                    fence_proxy_async_smem();
                    mbar_arrive(aready);
                } else {
                    // row (t, g) sees the writes of tokens s < t (s <= t when the read follows the write);
                    // A is masked, rounded to bfloat16 and handed back as an operand
                    if (np > 0) ST_WAIT(pfree, np - 1, 70);  // the last tile's A products are complete
                    tc_fence_after();
                    if (G > 0 && cq * 16 < Tc) {
                        float av[16];
                        const uint32_t abase = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + kColA + cq * 16;
                        tmem_ld16(abase, av);
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            const int c = cq * 2 + j;
                            float z[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                const int s = c * 8 + e;
                                const bool seen = is_read && (a.wtr ? s <= my_t : s < my_t);
                                z[e] = seen ? av[8 * j + e] : 0.f;
                            }
                            *reinterpret_cast<uint4*>(plo + r * 128 + ((c ^ sw) * 16)) = Chunk<__nv_bfloat16>::pack(z);
                        }
                    }
                    tc_fence_before();
                    fence_proxy_async_smem();
                    mbar_arrive(aready);
                }

                // ---- epilogue: this row's outputs (this thread: 32 of the 128 d), normalised by the row sum ----
                ST_WAIT(oready, qn, 67);
                tc_fence_after();
                // the row sum of a read row: its four quarters' sums of numerators (the residual operand is free again)
                float inv_l = 1.f;
                if (G > 0) {
                    rowstat[cq * 128 + r] = lr;
                    st_sync();
                    inv_l = 1.f / ((rowstat[r] + rowstat[128 + r]) + (rowstat[256 + r] + rowstat[384 + r]));
                    st_sync();
                }
                if (G > 0) {
                    const size_t orow = (((size_t)b * a.T + t0 + my_t) * a.Hq + (size_t)h * G + my_g) * 128 + cq * 32;
                    float o[32];
                    tmem_ld32(lane_base + kColO, o);
                    // (a ragged last chunk has rows past the last token: nothing is stored for them)
                    if (is_read && a.out != nullptr && t0 + my_t < a.T && !*abort_flag) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] *= inv_l;
                        if (a.out_f32) {
                            float4* dst = reinterpret_cast<float4*>(a.out + orow * 4);
#pragma unroll
                            for (int j = 0; j < 8; ++j) dst[j] = make_float4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
                        } else {
                            uint4* dst = reinterpret_cast<uint4*>(a.out + orow * 2);
#pragma unroll
                            for (int j = 0; j < 4; ++j) dst[j] = Chunk<__nv_bfloat16>::pack(o + 8 * j);
                        }
                    }
                }
                tc_fence_before();
                mbar_arrive(qfree);  // the chunk's operands and accumulators may be reused
            }
        }
    }
#undef ST_WAIT

    tc_fence_before();
    __syncthreads();
    if (warp == kStRowWarps + 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

using StKernelFn = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap,
                            const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const StArgs);

StKernelFn pick_stream(int G) {
    switch (G) {
        case 0: return stream_tc_kernel<0>;  // the write-only form
        case 1: return stream_tc_kernel<1>;
        case 2: return stream_tc_kernel<2>;
        case 3: return stream_tc_kernel<3>;
        case 4: return stream_tc_kernel<4>;
        case 5: return stream_tc_kernel<5>;
        case 6: return stream_tc_kernel<6>;
        case 7: return stream_tc_kernel<7>;
        default: return nullptr;
    }
}

// Step vectors [B][T][H][128] bfloat16 as a 4-D tensor (d, head, token, sequence); one box is
// 64 columns x `heads` heads x `tokens` tokens, landing as rows (token, head) with the 128-byte swizzle.
bool make_step_map(CUtensorMap* map, const void* base, int B, int T, int H, int heads, int tokens) {
    TensorMapEncodeFn fn = tensor_map_encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[4] = {128, (cuuint64_t)H, (cuuint64_t)T, (cuuint64_t)B};
    const cuuint64_t strides[3] = {256, (cuuint64_t)H * 256, (cuuint64_t)T * H * 256};
    const cuuint32_t box[4] = {64, (cuuint32_t)heads, (cuuint32_t)tokens, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// [U][C][128] bfloat16 plane as (d, slot, unit) with boxes of 64 columns x `rows` slots: the map
// the fill phase appends a chunk's keys and values through.
bool make_append_map(CUtensorMap* map, void* base, int U, int C, int rows) {
    TensorMapEncodeFn fn = tensor_map_encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[3] = {128, (cuuint64_t)C, (cuuint64_t)U};
    const cuuint64_t strides[2] = {256, (cuuint64_t)C * 256};
    const cuuint32_t box[3] = {64, (cuuint32_t)rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

int stream_chunk_tokens(const bct_cache* c) {
    const bct_params_t& p = c->p;
    if (p.dtype != BCT_BF16 || p.head_dim != 128 || c->G > 7 || !c->tc_ready) return 0;
    if (p.flags & BCT_FLAG_CUDA_CORES) return 0;
    if (p.capacity < kStTile || p.capacity > kStMaxCapacity) return 0;
    if (c->plane_bytes < (size_t)1 << 18) return 0;
    // as many tokens as leave the chunk's G*Tc read rows + Tc write rows (padded to 16) within 128 operand rows,
    // with the read rows a multiple of 8
    switch (c->G) {
        case 1: return 64;
        case 2: return 40;
        case 3: return 32;
        case 4: return 24;
        default: return 16;
    }
}

int launch_stream_tc(const bct_cache* c, const void* q, const void* k, const void* v, void* out, int64_t T,
                     const float* eta, int64_t t_begin, int64_t n_chunks, int fill_len, int write_only, int tc_tokens,
                     cudaStream_t stream, cudaError_t* err) {
    const bct_params_t& p = c->p;
    // write_only: the form without read queries (Algorithm 1's UpdateKV); tc_tokens: tokens per chunk
    // (0: the cache's default; a shorter chunk serves the ragged end of a call)
    const int G = write_only ? 0 : c->G;
    StKernelFn fn = pick_stream(G);
    const int Tc_max = write_only ? 128 : stream_chunk_tokens(c);
    const int Tc = tc_tokens > 0 ? tc_tokens : Tc_max;
    if (fn == nullptr || Tc_max == 0 || stream_chunk_tokens(c) == 0 || T > (int64_t)1 << 30 || Tc % 8 != 0 || Tc > Tc_max ||
        (write_only && fill_len >= 0) || (write_only && Tc % 16 != 0)) {
        *err = cudaErrorInvalidConfiguration;
        return -1;
    }
    if (fill_len >= 0 && fill_len + n_chunks * Tc > p.capacity) {
        *err = cudaErrorInvalidValue;
        return -1;
    }
    alignas(64) CUtensorMap mq, mk, mv, mka, mva;
    if (!make_append_map(&mka, c->kplane, c->U, p.capacity, Tc) || !make_append_map(&mva, c->vhi, c->U, p.capacity, Tc) ||
        !make_step_map(&mq, write_only ? k : q, p.batch, (int)T, write_only ? p.n_kv_heads : p.n_q_heads,
                       write_only ? 1 : c->G, Tc) ||
        !make_step_map(&mk, k, p.batch, (int)T, p.n_kv_heads, 1, Tc) ||
        !make_step_map(&mv, v, p.batch, (int)T, p.n_kv_heads, 1, Tc)) {
        *err = cudaErrorInvalidValue;
        return -1;
    }
    StArgs a;
    a.out = static_cast<char*>(out);
    a.status = c->status;
    a.eta = eta;
    a.C = p.capacity;
    a.Hq = p.n_q_heads;
    a.Hkv = p.n_kv_heads;
    a.U = c->U;
    a.T = (int)T;
    a.t_begin = (int)t_begin;
    a.n_chunks = (int)n_chunks;
    a.Tc = Tc;
    a.fill = fill_len >= 0 ? 1 : 0;
    a.len0 = fill_len >= 0 ? fill_len : 0;
    a.wtr = (p.flags & BCT_FLAG_WRITE_THEN_READ) ? 1 : 0;
    a.out_f32 = (p.flags & BCT_FLAG_OUT_F32) ? 1 : 0;
    a.precise = (p.flags & BCT_FLAG_PRECISE_READ) ? 1 : 0;
    a.read_scale = p.read_scale;
    a.write_scale = p.write_scale;
    a.write_eps = (p.flags & BCT_FLAG_DENSE_WRITE) ? 0.f : p.write_eps;
    const int smem = st_smem(Tc > kStMaxTc).total;
    *err = cudaFuncSetAttribute(reinterpret_cast<const void*>(fn), cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (*err != cudaSuccess) return -1;
    const int grid = c->U < c->sm_count ? c->U : c->sm_count;
    // Chunk-major dealing of the (unit, chunk) pairs where it saves a turn: units that do not divide by the CTAs, more
    // than one chunk, and no single-tile cache (which stays in one CTA's shared memory from chunk to chunk).
    const bool resident = fill_len < 0 && p.capacity <= kStTile && n_chunks > 1;
    const int64_t turns_unit_major = ((c->U + grid - 1) / grid) * n_chunks;
    const int64_t turns_chunk_major = ((int64_t)c->U * n_chunks + grid - 1) / grid;
    a.chunk_major = (!resident && c->U >= grid && n_chunks > 1 && turns_chunk_major < turns_unit_major) ? 1 : 0;
    a.progress = c->progress;
    a.launch = ++c->stream_launches;
    if (a.chunk_major) {
        // CTAs wait for one another here (a chunk for the unit's chunk before it, on another CTA), so every CTA of the
        // grid must be resident: a cooperative launch, which the runtime refuses when the grid does not fit the device
        // as it is (SMs held by other work, a partitioned device).  Refused: the unit-major walk, which waits for nobody.
        CUtensorMap tk = *reinterpret_cast<const CUtensorMap*>(c->tmap_k), tv = *reinterpret_cast<const CUtensorMap*>(c->tmap_v),
                    tl = *reinterpret_cast<const CUtensorMap*>(c->tmap_lo);
        void* args[] = {&tk, &tv, &tl, &mq, &mk, &mv, &mka, &mva, &a};
        *err = cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(fn), dim3(grid), dim3(kStThreads), args, (size_t)smem, stream);
        if (*err == cudaSuccess) return 1;
        (void)cudaGetLastError();
        a.chunk_major = 0;
    }
    fn<<<grid, kStThreads, smem, stream>>>(*reinterpret_cast<const CUtensorMap*>(c->tmap_k),
                                           *reinterpret_cast<const CUtensorMap*>(c->tmap_v),
                                           *reinterpret_cast<const CUtensorMap*>(c->tmap_lo), mq, mk, mv, mka, mva, a);
    *err = cudaGetLastError();
    return *err == cudaSuccess ? 1 : -1;
}

}  // namespace bct
