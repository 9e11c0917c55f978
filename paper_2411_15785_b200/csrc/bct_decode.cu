// Fused decode step of the bounded-cache attention layer for sm_100a.
//
// One thread-block cluster of S CTAs serves one (sequence, kv-head) unit; each CTA owns
// a contiguous slice of the C slots.  Per token the CTA
//   1. streams its slice of MK once through a shared-memory ring (TMA-engine bulk
//      copies, mbarrier hand-off) and forms, per slot, the G read scores and the write
//      score  score_t = wq_t . MK^T  (Algorithm 1),
//   2. turns them into softmax numerators; the write row's maximum and sum are
//      exchanged across the cluster so that ww_t = softmax(score_t) is normalised over
//      all C slots before any slot is rewritten,
//   3. streams its slice of MV once through the same ring, accumulates the G attention
//      outputs from MV_{t-1} and applies  MV_t = MV_{t-1} + ww_t^T . wv_t  (Method step 4)
//      to the slots whose weight reaches write_eps, storing only those rows,
//   4. merges the per-CTA partial outputs (online-softmax combine) in CTA 0.
// While the cache is filling (len < C) the token is appended at slot len instead and
// the read covers the resident slots including the appended one.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "bct_device.cuh"
#include "bct_internal.h"

namespace bct {
namespace {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;  // + one producer warp
constexpr int kTileBytes = 16384;
constexpr int kStages = 4;
constexpr int kMaxCluster = 8;
constexpr float kNegBig = -3.0e38f;

struct DecodeArgs {
    const char* kplane;
    char* vhi;
    char* vlo;
    const char* q;
    const char* k;
    const char* v;
    char* out;
    int* status;
    long long q_bs;   // elements between sequences in q / out
    long long kv_bs;  // elements between sequences in k / v
    const float* eta; // step size of each unit's write, [sequence][kv-head], or NULL (all ones)
    long long eta_bs; // elements between sequences in eta
    int C;
    int len;         // resident slots before this token
    int slice_rows;  // slots per CTA of the cluster
    int S;           // cluster size
    int Hkv;
    int score_stride;
    int do_write;  // the soft write happens this token
    int wtr;       // the read sees the token's own write
    int dense;     // rewrite every slot
    int out_f32;   // out is float whatever the cache dtype
    int precise;   // bfloat16 cache: the read uses value + residual (streams the residual plane too)
    float read_scale;
    float write_scale;
    float write_eps;
};

// Shared-memory carve-up, the same on host and device.
struct SmemLayout {
    int ring, scores, red, stat, wstat, merge, bars, total;
};
__host__ __device__ inline SmemLayout smem_layout(int G, int D, int score_stride, int S) {
    SmemLayout L;
    int off = 0;
    L.ring = off;
    off += kStages * kTileBytes;
    L.scores = off;
    off += (G + 1) * score_stride * 4;
    L.red = off;
    off += kConsumerWarps * (G + 1) * 4;
    L.stat = off;
    off += 2 * (G + 1) * 4 + 16;
    L.wstat = off;
    off += kMaxCluster * 2 * 4;
    L.merge = off;
    off += (S > 1 ? (S - 1) * G * (D + 3) * 4 : 0);
    off = (off + 15) & ~15;
    L.bars = off;
    off += (2 * kStages + 1) * 8;
    L.total = (off + 127) & ~127;
    return L;
}

__device__ __forceinline__ void consumer_sync() {
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
}

// out has the layout of q; q_off is the unit's byte offset in q's element size.
template <typename T>
__device__ __forceinline__ void store_out(const DecodeArgs& a, size_t q_off, int idx, float val) {
    if (a.out_f32)
        reinterpret_cast<float*>(a.out + q_off / sizeof(T) * sizeof(float))[idx] = val;
    else
        reinterpret_cast<T*>(a.out + q_off)[idx] = (T)val;
}

template <typename T, int D, int G>
__global__ void __launch_bounds__(kThreads, (G <= 4 ? 2 : 1)) decode_kernel(const DecodeArgs a) {
    using Ck = Chunk<T>;
    constexpr int EPL = Ck::kElems;                // elements per 16-byte chunk
    constexpr int ROW_BYTES = D * (int)sizeof(T);  // one cache row
    constexpr int LPR = ROW_BYTES / 16;            // lanes sharing a row
    constexpr int RPW = 32 / LPR;                  // rows a warp covers per pass
    constexpr int TILE_ROWS = kTileBytes / ROW_BYTES;
    constexpr int ROWS_PER_PASS = kConsumerWarps * RPW;
    constexpr int PASSES = TILE_ROWS / ROWS_PER_PASS;
    static_assert(LPR >= 1 && LPR <= 32 && (32 % LPR) == 0, "row must split into 1..32 chunks");
    static_assert(TILE_ROWS % ROWS_PER_PASS == 0, "tile must be a whole number of passes");

    extern __shared__ __align__(128) unsigned char smem[];
    const int S = a.S;
    const SmemLayout L = smem_layout(G, D, a.score_stride, S);
    unsigned char* ring = smem + L.ring;
    float* sc = reinterpret_cast<float*>(smem + L.scores);
    float* red = reinterpret_cast<float*>(smem + L.red);
    float* stat = reinterpret_cast<float*>(smem + L.stat);  // m[G+1], l[G+1], abort flag
    volatile int* abort_flag = reinterpret_cast<volatile int*>(stat + 2 * (G + 1));
    float* wstat = reinterpret_cast<float*>(smem + L.wstat);
    float* merge = reinterpret_cast<float*>(smem + L.merge);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L.bars);
    uint64_t* empty = full + kStages;
    uint64_t* xbar = empty + kStages;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const int rank = (S > 1) ? (int)cluster_ctarank() : 0;
    const int u = blockIdx.x / S;
    const int b = u / a.Hkv;
    const int h_kv = u - b * a.Hkv;
    const int stride = a.score_stride;

    // this CTA's slice of the slots
    const int slice_start = rank * a.slice_rows;
    const int n_slice = max(0, min(a.slice_rows, a.C - slice_start));
    const int n_stream = max(0, min(a.len - slice_start, n_slice));  // rows that come from the cache
    const bool has_virtual = (a.len < a.C) && (a.len >= slice_start) && (a.len < slice_start + n_slice);
    const int n_rows = n_stream + (has_virtual ? 1 : 0);
    const int nt = (n_stream + TILE_ROWS - 1) / TILE_ROWS;

    const size_t unit_off = (size_t)u * a.C * ROW_BYTES;
    const char* kslice = a.kplane + unit_off + (size_t)slice_start * ROW_BYTES;
    char* vslice = a.vhi + unit_off + (size_t)slice_start * ROW_BYTES;
    const bool precise = (sizeof(T) == 2) && a.precise;
    const size_t q_off = ((size_t)b * a.q_bs + (size_t)h_kv * G * D) * sizeof(T);
    const size_t kv_off = ((size_t)b * a.kv_bs + (size_t)h_kv * D) * sizeof(T);
    // step size of this token's write: MV_t = MV_{t-1} + eta_t ww_t^T wv_t (the write value is scaled once)
    const float eta_u = (a.eta != nullptr && a.do_write) ? a.eta[(size_t)b * a.eta_bs + h_kv] : 1.f;

    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(&full[i], 1);
            mbar_init(&empty[i], kConsumerWarps);
        }
        mbar_init(xbar, S);
        *abort_flag = 0;
        fence_mbar_init_cluster();
    }
    __syncthreads();
    if (S > 1) {  // every CTA of the cluster is running and its barriers exist
        cluster_arrive();
        cluster_wait();
    }

    if (warp == kConsumerWarps) {
        // ---------------- producer warp: K tiles, then V tiles, through the ring ----------------
        if (lane == 0) {
            const char* loslice = precise ? a.vlo + unit_off + (size_t)slice_start * ROW_BYTES : nullptr;
            const int n_items = precise ? 3 * nt : 2 * nt;  // K tiles, then V tiles (value, residual interleaved)
            for (int item = 0; item < n_items; ++item) {
                const int stage = item % kStages;
                if (item >= kStages) {
                    const uint32_t parity = ((item / kStages) - 1) & 1;
                    if (!mbar_wait_abortable(&empty[stage], parity, abort_flag)) {
                        report_timeout(a.status, 1);
                        *abort_flag = 1;
                        break;
                    }
                }
                int t = item;
                const char* base = kslice;
                if (item >= nt) {
                    const int j = item - nt;
                    t = precise ? (j >> 1) : j;
                    base = (precise && (j & 1)) ? loslice : (const char*)vslice;
                }
                const int rows = min(TILE_ROWS, n_stream - t * TILE_ROWS);
                const char* src = base + (size_t)t * kTileBytes;
                const uint32_t bytes = (uint32_t)rows * ROW_BYTES;
                mbar_arrive_expect_tx(&full[stage], bytes);
                bulk_load(ring + stage * kTileBytes, src, bytes, &full[stage]);
            }
        }
        __syncwarp();
    } else {
        // ---------------- consumer warps ----------------
        const int chunk = lane % LPR;  // which 16 bytes of the row
        const int sub = lane / LPR;    // which row of the warp's pass

        // step vectors of this unit: G read queries (pre-scaled) and the write query
        float qreg[G + 1][EPL];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const uint4 w = *reinterpret_cast<const uint4*>(a.q + q_off + (size_t)g * ROW_BYTES + chunk * 16);
            Ck::unpack(w, qreg[g]);
#pragma unroll
            for (int e = 0; e < EPL; ++e) qreg[g][e] *= a.read_scale;
        }
        const uint4 k_raw = *reinterpret_cast<const uint4*>(a.k + kv_off + chunk * 16);
        const uint4 v_raw = *reinterpret_cast<const uint4*>(a.v + kv_off + chunk * 16);
        Ck::unpack(k_raw, qreg[G]);
#pragma unroll
        for (int e = 0; e < EPL; ++e) qreg[G][e] *= a.write_scale;

        // ---- phase K: scores of every resident slot of the slice ----
        for (int i = 0; i < nt; ++i) {
            const int stage = i % kStages;
            if (!mbar_wait_abortable(&full[stage], (i / kStages) & 1, abort_flag)) {
                report_timeout(a.status, 2);
                *abort_flag = 1;
            }
            const int rows = min(TILE_ROWS, n_stream - i * TILE_ROWS);
            const unsigned char* tile = ring + stage * kTileBytes;
            uint4 w[PASSES];
#pragma unroll
            for (int ps = 0; ps < PASSES; ++ps) {
                const int r = ps * ROWS_PER_PASS + warp * RPW + sub;
                w[ps] = (r < rows) ? *reinterpret_cast<const uint4*>(tile + r * ROW_BYTES + chunk * 16)
                                   : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int ps = 0; ps < PASSES; ++ps) {
                const int r = ps * ROWS_PER_PASS + warp * RPW + sub;
                float x[EPL];
                Ck::unpack(w[ps], x);
                float acc[G + 1];
#pragma unroll
                for (int h = 0; h <= G; ++h) {
                    float s = 0.f;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) s = fmaf(qreg[h][e], x[e], s);
                    acc[h] = s;
                }
#pragma unroll
                for (int h = 0; h <= G; ++h) {
#pragma unroll
                    for (int o = LPR / 2; o > 0; o >>= 1) acc[h] += __shfl_xor_sync(0xffffffffu, acc[h], o);
                }
                if (chunk == 0 && r < rows) {
#pragma unroll
                    for (int h = 0; h <= G; ++h) sc[h * stride + i * TILE_ROWS + r] = acc[h];
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[stage]);
        }

        // ---- fill phase: the appended slot is scored from the step vectors and stored ----
        if (has_virtual && warp == 0) {
            float kx[EPL];
            Ck::unpack(k_raw, kx);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float s = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; ++e) s = fmaf(qreg[g][e], kx[e], s);
#pragma unroll
                for (int o = LPR / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                if (lane == 0) sc[g * stride + n_stream] = s;
            }
            if (sub == 0) {
                const size_t off = unit_off + (size_t)a.len * ROW_BYTES + chunk * 16;
                *reinterpret_cast<uint4*>(const_cast<char*>(a.kplane) + off) = k_raw;
                *reinterpret_cast<uint4*>(a.vhi + off) = v_raw;
                if (a.vlo) *reinterpret_cast<uint4*>(a.vlo + off) = make_uint4(0, 0, 0, 0);
            }
        }
        consumer_sync();

        // ---- softmax numerators in place: row maxima, then exp and row sums ----
        const int n_heads = a.do_write ? G + 1 : G;  // the write row only when a write follows
        {
            float mx[G + 1];
#pragma unroll
            for (int h = 0; h <= G; ++h) mx[h] = kNegBig;
            for (int j = tid; j < n_rows; j += kConsumerThreads) {
#pragma unroll
                for (int h = 0; h <= G; ++h)
                    if (h < n_heads) mx[h] = fmaxf(mx[h], sc[h * stride + j]);
            }
#pragma unroll
            for (int h = 0; h <= G; ++h) {
                mx[h] = warp_max(mx[h]);
                if (lane == 0) red[warp * (G + 1) + h] = mx[h];
            }
            consumer_sync();
            if (tid <= G) {
                float m = kNegBig;
                for (int w2 = 0; w2 < kConsumerWarps; ++w2) m = fmaxf(m, red[w2 * (G + 1) + tid]);
                stat[tid] = m;
            }
            consumer_sync();
            float sm[G + 1];
#pragma unroll
            for (int h = 0; h <= G; ++h) sm[h] = 0.f;
            for (int j = tid; j < n_rows; j += kConsumerThreads) {
#pragma unroll
                for (int h = 0; h <= G; ++h)
                    if (h < n_heads) {
                        const float e = __expf(sc[h * stride + j] - stat[h]);
                        sc[h * stride + j] = e;
                        sm[h] += e;
                    }
            }
#pragma unroll
            for (int h = 0; h <= G; ++h) {
                sm[h] = warp_sum(sm[h]);
                if (lane == 0) red[warp * (G + 1) + h] = sm[h];
            }
            consumer_sync();
            if (tid <= G) {
                float l = 0.f;
                for (int w2 = 0; w2 < kConsumerWarps; ++w2) l += red[w2 * (G + 1) + tid];
                stat[(G + 1) + tid] = l;
            }
            consumer_sync();
        }

        // ---- write weights need the maximum and sum over ALL C slots: cluster exchange ----
        float wfac = 0.f;  // ww_j = numerator_j * wfac
        if (a.do_write) {
            if (S > 1) {
                if (tid == 0) {
                    for (int r = 0; r < S; ++r) {
                        const uint32_t dst = map_to_rank(wstat + 2 * rank, r);
                        st_cluster_f32(dst, stat[G]);
                        st_cluster_f32(dst + 4, stat[(G + 1) + G]);
                        mbar_arrive_remote(map_to_rank(xbar, r));
                    }
                }
                if (!mbar_wait_abortable<true>(xbar, 0, abort_flag)) {
                    report_timeout(a.status, 3);
                    *abort_flag = 1;
                }
                float M = kNegBig;
                for (int r = 0; r < S; ++r) M = fmaxf(M, wstat[2 * r]);
                float Lsum = 0.f;
                for (int r = 0; r < S; ++r) Lsum += wstat[2 * r + 1] * __expf(wstat[2 * r] - M);
                wfac = __expf(stat[G] - M) / Lsum;
            } else {
                wfac = 1.f / stat[(G + 1) + G];
            }
        }

        // ---- phase V: outputs from MV_{t-1}, then the update rule on the rows it changes ----
        float o[G][EPL];
        float wd[G];  // sum_j p_j * ww_j, for the write-then-read order
#pragma unroll
        for (int g = 0; g < G; ++g) {
            wd[g] = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) o[g][e] = 0.f;
        }
        float vt[EPL];
        Ck::unpack(v_raw, vt);
#pragma unroll
        for (int e = 0; e < EPL; ++e) vt[e] *= eta_u;
        int rows_stored = 0;  // rows of MV this thread's row group rewrites (counted by the lane of chunk 0)
        for (int i = 0; i < nt; ++i) {
            const int item = precise ? nt + 2 * i : nt + i;
            const int stage = item % kStages;
            if (!mbar_wait_abortable(&full[stage], (item / kStages) & 1, abort_flag)) {
                report_timeout(a.status, 4);
                *abort_flag = 1;
            }
            const int stage_lo = (item + 1) % kStages;
            if (precise && !mbar_wait_abortable(&full[stage_lo], ((item + 1) / kStages) & 1, abort_flag)) {
                report_timeout(a.status, 5);
                *abort_flag = 1;
            }
            const int rows = min(TILE_ROWS, n_stream - i * TILE_ROWS);
            const unsigned char* tile = ring + stage * kTileBytes;
            const unsigned char* tile_lo = ring + stage_lo * kTileBytes;
            uint4 w[PASSES];
#pragma unroll
            for (int ps = 0; ps < PASSES; ++ps) {
                const int r = ps * ROWS_PER_PASS + warp * RPW + sub;
                w[ps] = (r < rows) ? *reinterpret_cast<const uint4*>(tile + r * ROW_BYTES + chunk * 16)
                                   : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int ps = 0; ps < PASSES; ++ps) {
                const int r = ps * ROWS_PER_PASS + warp * RPW + sub;
                if (r < rows) {
                    const int row = i * TILE_ROWS + r;
                    float x[EPL];
                    Ck::unpack(w[ps], x);
                    float lo[EPL];
                    if constexpr (sizeof(T) == 2) {
                        if (precise) {
                            Ck::unpack(*reinterpret_cast<const uint4*>(tile_lo + r * ROW_BYTES + chunk * 16), lo);
#pragma unroll
                            for (int e = 0; e < EPL; ++e) x[e] += lo[e];  // exact: <= 17 significant bits
                        }
                    }
                    float p[G];
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        p[g] = sc[g * stride + row];
#pragma unroll
                        for (int e = 0; e < EPL; ++e) o[g][e] = fmaf(p[g], x[e], o[g][e]);
                    }
                    if (a.do_write) {
                        const float ww = sc[G * stride + row] * wfac;
                        if (a.dense || ww >= a.write_eps) {
                            // (a read that follows its own write sees the rows actually rewritten)
#pragma unroll
                            for (int g = 0; g < G; ++g) wd[g] = fmaf(p[g], ww, wd[g]);
                            if (chunk == 0) ++rows_stored;
                            const size_t off = (size_t)row * ROW_BYTES + chunk * 16;
                            float nv[EPL];
                            if constexpr (sizeof(T) == 2) {
                                char* lo_ptr = a.vlo + unit_off + (size_t)slice_start * ROW_BYTES + off;
                                if (!precise) {
                                    Ck::unpack(*reinterpret_cast<const uint4*>(lo_ptr), lo);
#pragma unroll
                                    for (int e = 0; e < EPL; ++e) x[e] += lo[e];
                                }
#pragma unroll
                                for (int e = 0; e < EPL; ++e) nv[e] = fmaf(ww, vt[e], x[e]);
                                const uint4 hi_new = Ck::pack(nv);
                                float hf[EPL];
                                Ck::unpack(hi_new, hf);
#pragma unroll
                                for (int e = 0; e < EPL; ++e) nv[e] -= hf[e];
                                *reinterpret_cast<uint4*>(vslice + off) = hi_new;
                                *reinterpret_cast<uint4*>(lo_ptr) = Ck::pack(nv);
                            } else {
#pragma unroll
                                for (int e = 0; e < EPL; ++e) nv[e] = fmaf(ww, vt[e], x[e]);
                                *reinterpret_cast<uint4*>(vslice + off) = Ck::pack(nv);
                            }
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&empty[stage]);
                if (precise) mbar_arrive(&empty[stage_lo]);
            }
        }
        rows_stored = __reduce_add_sync(0xffffffffu, rows_stored);
        if (lane == 0 && rows_stored > 0)
            atomicAdd(reinterpret_cast<unsigned long long*>(a.status + kStatusRowsWord), (unsigned long long)rows_stored);
        if (has_virtual && warp == 0 && sub == 0) {  // the appended slot's own value row
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float p = sc[g * stride + n_stream];
#pragma unroll
                for (int e = 0; e < EPL; ++e) o[g][e] = fmaf(p, vt[e], o[g][e]);
            }
        }

        // ---- reduce the partial outputs over the rows of a pass, then over the warps ----
#pragma unroll
        for (int g = 0; g < G; ++g) {
#pragma unroll
            for (int ofs = LPR; ofs < 32; ofs <<= 1) {
                wd[g] += __shfl_xor_sync(0xffffffffu, wd[g], ofs);
#pragma unroll
                for (int e = 0; e < EPL; ++e) o[g][e] += __shfl_xor_sync(0xffffffffu, o[g][e], ofs);
            }
        }
        consumer_sync();                                    // every warp is done with the ring
        float* ored = reinterpret_cast<float*>(ring);       // [warp][G][D+1]
        float* ofin = ored + kConsumerWarps * G * (D + 1);  // [G][D+1]
        if (sub == 0) {
#pragma unroll
            for (int g = 0; g < G; ++g) {
#pragma unroll
                for (int e = 0; e < EPL; ++e) ored[(warp * G + g) * (D + 1) + chunk * EPL + e] = o[g][e];
                if (lane == 0) ored[(warp * G + g) * (D + 1) + D] = wd[g];
            }
        }
        consumer_sync();
        for (int idx = tid; idx < G * (D + 1); idx += kConsumerThreads) {
            float s = 0.f;
#pragma unroll
            for (int w2 = 0; w2 < kConsumerWarps; ++w2) s += ored[w2 * G * (D + 1) + idx];
            ofin[idx] = s;
        }
        consumer_sync();

        const bool add_own = a.wtr && a.do_write;
        if (S == 1) {
            if (a.out != nullptr && !*abort_flag) {
                const T* vin = reinterpret_cast<const T*>(a.v + kv_off);
                for (int idx = tid; idx < G * D; idx += kConsumerThreads) {
                    const int g = idx / D, e = idx - g * D;
                    const float inv = 1.f / stat[(G + 1) + g];
                    float val = ofin[g * (D + 1) + e] * inv;
                    if (add_own) val = fmaf(ofin[g * (D + 1) + D] * inv, (float)vin[e] * eta_u, val);
                    store_out<T>(a, q_off, idx, val);
                }
            }
        } else if (rank != 0) {
            // hand the partial (numerators, max, sum) to CTA 0 of the cluster
            float* dst0 = merge + (size_t)(rank - 1) * G * (D + 3);
            for (int idx = tid; idx < G * (D + 3); idx += kConsumerThreads) {
                const int g = idx / (D + 3), e = idx - g * (D + 3);
                const float val = (e <= D) ? ofin[g * (D + 1) + e] : (e == D + 1 ? stat[g] : stat[(G + 1) + g]);
                st_cluster_f32(map_to_rank(dst0 + idx, 0), val);
            }
        }
    }

    if (S > 1) {
        // all partials have landed in CTA 0; nobody leaves while its memory may be written
        cluster_arrive();
        cluster_wait();
        if (rank == 0 && warp < kConsumerWarps && a.out != nullptr && !*abort_flag) {
            const float* ofin = reinterpret_cast<float*>(ring) + kConsumerWarps * G * (D + 1);
            const T* vin = reinterpret_cast<const T*>(a.v + kv_off);
            const bool add_own = a.wtr && a.do_write;
            for (int idx = tid; idx < G * D; idx += kConsumerThreads) {
                const int g = idx / D, e = idx - g * D;
                float M = stat[g];
                for (int r = 1; r < S; ++r) M = fmaxf(M, merge[((r - 1) * G + g) * (D + 3) + D + 1]);
                const float f0 = __expf(stat[g] - M);
                float num = ofin[g * (D + 1) + e] * f0;
                float own = ofin[g * (D + 1) + D] * f0;
                float den = stat[(G + 1) + g] * f0;
                for (int r = 1; r < S; ++r) {
                    const float* mr = merge + ((r - 1) * G + g) * (D + 3);
                    const float f = __expf(mr[D + 1] - M);
                    num = fmaf(mr[e], f, num);
                    own = fmaf(mr[D], f, own);
                    den = fmaf(mr[D + 2], f, den);
                }
                float val = num / den;
                if (add_own) val = fmaf(own / den, (float)vin[e] * eta_u, val);
                store_out<T>(a, q_off, idx, val);
            }
        }
    }
}

using KernelFn = void (*)(const DecodeArgs);

template <typename T, int D>
KernelFn pick_group(int G) {
    switch (G) {
        case 1: return decode_kernel<T, D, 1>;
        case 2: return decode_kernel<T, D, 2>;
        case 3: return decode_kernel<T, D, 3>;
        case 4: return decode_kernel<T, D, 4>;
        case 5: return decode_kernel<T, D, 5>;
        case 6: return decode_kernel<T, D, 6>;
        case 7: return decode_kernel<T, D, 7>;
        case 8: return decode_kernel<T, D, 8>;
        default: return nullptr;
    }
}

KernelFn pick_kernel(int dtype, int D, int G) {
    if (dtype == BCT_F32) {
        if (D == 64) return pick_group<float, 64>(G);
        if (D == 128) return pick_group<float, 128>(G);
    } else if (dtype == BCT_BF16) {
        if (D == 64) return pick_group<__nv_bfloat16, 64>(G);
        if (D == 128) return pick_group<__nv_bfloat16, 128>(G);
    }
    return nullptr;
}

// Cluster size and slice length for a capacity: the smallest cluster whose per-CTA
// score array leaves room for two CTAs per SM, widened while the grid would leave SMs idle.
struct Plan {
    int S, slice_rows, score_stride, smem;
    bool ok;
};
Plan make_plan(int G, int D, int elem_bytes, int C, int U, int sm_count, int smem_optin) {
    Plan best{0, 0, 0, 0, false};
    const int tile_rows = kTileBytes / (D * elem_bytes);
    const int two_per_sm = (smem_optin + 1024) / 2 - 1024;
    for (int pass = 0; pass < 2 && !best.ok; ++pass) {
        const int limit = pass == 0 ? two_per_sm : smem_optin;
        for (int S = 1; S <= kMaxCluster; S *= 2) {
            const int slice = (C + S - 1) / S;
            const int stride = (slice + 3) & ~3;
            const int smem = smem_layout(G, D, stride, S).total;
            if (smem <= limit) {
                best = Plan{S, slice, stride, smem, true};
                break;
            }
        }
    }
    if (!best.ok) return best;
    // widen for small grids: keep at least one tile per CTA
    while (best.S < kMaxCluster && (long long)U * best.S < 2LL * sm_count) {
        const int S = best.S * 2;
        const int slice = (C + S - 1) / S;
        if (slice < tile_rows) break;
        const int stride = (slice + 3) & ~3;
        best = Plan{S, slice, stride, smem_layout(G, D, stride, S).total, true};
    }
    return best;
}

}  // namespace

bool decode_supported(const bct_params_t& p, int smem_optin, const char** why) {
    const int G = p.n_q_heads / p.n_kv_heads;
    if (pick_kernel(p.dtype, p.head_dim, G) == nullptr) {
        *why = "no decode kernel for this dtype / head_dim / group size (head_dim in {64,128}, group <= 8)";
        return false;
    }
    Plan pl = make_plan(G, p.head_dim, p.dtype == BCT_F32 ? 4 : 2, p.capacity, p.batch * p.n_kv_heads, 148,
                        smem_optin);
    if (!pl.ok) {
        *why = "capacity * (group + 1) too large for the shared-memory score array of an 8-CTA cluster";
        return false;
    }
    return true;
}

int launch_decode(const bct_cache* c, const StepIO& io, int len, int do_write, cudaStream_t stream,
                  cudaError_t* err) {
    const bct_params_t& p = c->p;
    if (!(p.flags & BCT_FLAG_CUDA_CORES) && tc_eligible(c)) return launch_decode_tc(c, io, len, do_write, stream, err);
    KernelFn fn = pick_kernel(p.dtype, p.head_dim, c->G);
    Plan pl = make_plan(c->G, p.head_dim, c->elem_bytes, p.capacity, c->U, c->sm_count, c->smem_optin);
    if (fn == nullptr || !pl.ok) {
        *err = cudaErrorInvalidConfiguration;
        return -1;
    }
    DecodeArgs a;
    a.kplane = c->kplane;
    a.vhi = c->vhi;
    a.vlo = c->vlo;
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
    a.slice_rows = pl.slice_rows;
    a.S = pl.S;
    a.Hkv = p.n_kv_heads;
    a.score_stride = pl.score_stride;
    a.do_write = (len == p.capacity) && do_write;
    a.wtr = (p.flags & BCT_FLAG_WRITE_THEN_READ) ? 1 : 0;
    a.dense = (p.flags & BCT_FLAG_DENSE_WRITE) ? 1 : 0;
    a.out_f32 = (p.flags & BCT_FLAG_OUT_F32) ? 1 : 0;
    a.precise = (p.flags & BCT_FLAG_PRECISE_READ) ? 1 : 0;
    a.read_scale = p.read_scale;
    a.write_scale = p.write_scale;
    a.write_eps = p.write_eps;

    *err = cudaFuncSetAttribute(reinterpret_cast<const void*>(fn), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                pl.smem);
    if (*err != cudaSuccess) return -1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(c->U * pl.S), 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)pl.smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)pl.S;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    *err = cudaLaunchKernelEx(&cfg, fn, a);
    if (*err != cudaSuccess) return -1;
    return 1;
}

}  // namespace bct
