// The projections in front of the bounded-cache layer on the sm_100a tensor path.
//
// Algorithm 1 starts every token with two products, wq_t = W_wq x_t and wv_t = W_wv x_t (the first two
// statements of its loop body); the read query of the attention layer is a third product of the same token.  For a block of tokens they are one contraction
//     [q | k | v][m][n] = sum_c x[m][c] * W[n][c]        W = W_q, W_wq, W_wv stacked over n
// with bfloat16 operands, fp32 accumulation in tensor memory and bfloat16 results, written straight
// into the three step-vector arrays the layer reads.
//
// One persistent CTA per SM over 128 x BN output tiles (BN = 128 for blocks of tokens, 32 for a
// decode step, where the weights stream once from HBM and more, smaller tiles fill the SMs):
//   warp 0      producer : TMA loads of x and W tiles (64 columns = 128 bytes per row, 128-byte swizzle)
//                          into a ring of stages
//   warp 1      MMA      : tcgen05.mma (M = 128, N = BN, K = 16) four times per stage; its commit frees the
//                          stage; two accumulators in tensor memory, so that the epilogue of one tile
//                          overlaps the products of the next
//   warps 2-5   epilogue : one thread per output row: tcgen05.ld, round to bfloat16, 64-byte stores
// Rows past the last token and columns past d_model are zero-filled by the TMA unit (with fewer than
// 128 tokens the box of x is shorter and the rows below it are never read back).
// Every wait is bounded; a timeout sets the status word and the kernel runs to its end.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>
#include <mutex>

#include "bct_internal.h"
#include "bct_tc.cuh"

namespace bct {
namespace {

constexpr int kPjThreads = 192;
constexpr int kPjBM = 128;
constexpr int kPjBK = 64;                      // columns per stage: 128 bytes per row
constexpr int kPjABytes = kPjBM * kPjBK * 2;   // 16 KiB
constexpr int kPjMaxStages = 16;

struct PjArgs {
    __nv_bfloat16* out[3];   // q, k, v
    int* status;             // may be NULL (no cache at hand): timeouts are then only counted in the return path
    int n_seg[3];            // output features of each segment (multiples of BN)
    long long M;             // tokens
    int K;                   // d_model
    int stages;
    int a_rows;              // rows of x one TMA box brings (128, or fewer when there are fewer tokens)
    int a_bytes;             // a_rows * 128: the x part of a stage; the W part (BN * 128 bytes) follows it
};


__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}

template <int BN, int KPER>
__global__ void __launch_bounds__(kPjThreads, 1)
project_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW0,
               const __grid_constant__ CUtensorMap tmW1, const __grid_constant__ CUtensorMap tmW2, const PjArgs a) {
    extern __shared__ unsigned char pj_smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(pj_smem_raw) + 1023) & ~uintptr_t(1023));
    const int kBlock = a.a_bytes + BN * kPjBK * 2;  // one 64-column block: x part, then W part
    const int kStage = KPER * kBlock;               // small blocks travel several to a stage: fewer hand-overs
    constexpr uint32_t kTmemCols = (2 * BN < 32) ? 32 : 2 * BN;   // two accumulators (a power of two)
    unsigned char* ring = smem;
    // The MMA always reads 128 rows of x: with a shorter box the rows below it are whatever follows in
    // shared memory (their output rows are never stored), so the last stage is followed by that much padding.
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)a.stages * kStage + (kPjABytes - a.a_bytes));
    uint64_t* full = bars;                        // [stages] tile pair landed (TMA transaction bytes)
    uint64_t* empty = bars + kPjMaxStages;        // [stages] products that read the stage complete (commit)
    uint64_t* acc_full = bars + 2 * kPjMaxStages;     // [2] accumulator complete (commit)
    uint64_t* acc_empty = bars + 2 * kPjMaxStages + 2;  // [2] accumulator read out (128 arrivals)
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * kPjMaxStages + 4);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kPjMaxStages + 5);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const int m_tiles = (int)((a.M + kPjBM - 1) / kPjBM);
    const int nt0 = a.n_seg[0] / BN, nt1 = a.n_seg[1] / BN, nt2 = a.n_seg[2] / BN;
    const int n_tiles = (nt0 + nt1 + nt2) * m_tiles;
    const int kb_count = (a.K + kPjBK - 1) / kPjBK;

    if (tid == 0) {
        for (int i = 0; i < a.stages; ++i) {
            mbar_init(&full[i], 1);
            mbar_init(&empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&acc_full[i], 1);
            mbar_init(&acc_empty[i], 128);
        }
        *abort_flag = 0;
        fence_mbar_init_cluster();
    }
    if (warp == 1) tmem_alloc(tmem_slot, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

#define PJ_WAIT(bar, parity, site)                                      \
    if (!mbar_wait_abortable(bar, (parity) & 1, abort_flag)) {          \
        if (a.status != nullptr) report_timeout(a.status, site);        \
        *abort_flag = 1;                                                \
    }

    // tile id -> (segment, first feature of the tile within the segment, first token)
    auto locate = [&](int tile, int* seg, int* n0, int* m0) {
        const int nt = tile / m_tiles;
        *m0 = (tile - nt * m_tiles) * kPjBM;
        if (nt < nt0) {
            *seg = 0;
            *n0 = nt * BN;
        } else if (nt < nt0 + nt1) {
            *seg = 1;
            *n0 = (nt - nt0) * BN;
        } else {
            *seg = 2;
            *n0 = (nt - nt0 - nt1) * BN;
        }
    };

    if (warp == 0) {
        // =========================== producer ===========================
        if (lane == 0) {
            int s = 0;        // stage of the next load
            uint32_t ph = 0;  // parity of the ring pass: pass p waits for the commits of pass p - 1
            bool first_pass = true;
            for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
                int seg, n0, m0;
                locate(tile, &seg, &n0, &m0);
                const CUtensorMap* tw = seg == 0 ? &tmW0 : (seg == 1 ? &tmW1 : &tmW2);
                // every CTA starts its walk over d_model at another column block: otherwise all of them ask
                // L2 for the same lines of x at the same time
                const int kb0 = (int)(((unsigned)blockIdx.x * 5u + (unsigned)tile) % (unsigned)kb_count);
                // Column blocks are asked for in groups: a row of W is 128 bytes per block, and neighbouring
                // blocks requested together let one DRAM page visit serve several of them.
                for (int i0 = 0; i0 < kb_count; i0 += KPER) {
                    const int nblk = min(KPER, kb_count - i0);
                    if (!first_pass) PJ_WAIT(&empty[s], ph ^ 1u, 81);
                    mbar_arrive_expect_tx(&full[s], (uint32_t)(nblk * kBlock));
                    for (int j = 0; j < nblk; ++j) {
                        const int i = i0 + j;
                        const int kb = kb0 + i < kb_count ? kb0 + i : kb0 + i - kb_count;
                        unsigned char* dst = ring + (size_t)s * kStage + (size_t)j * kBlock;
                        tma_load_2d(dst + a.a_bytes, tw, kb * kPjBK, n0, &full[s]);
                        tma_load_2d(dst, &tmX, kb * kPjBK, m0, &full[s]);
                    }
                    if (++s == a.stages) {
                        s = 0;
                        ph ^= 1u;
                        first_pass = false;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // =========================== MMA issuer ===========================
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc_mn(128, BN, false, false);  // x tile (K-major) x W tile (K-major)
            uint32_t nacc = 0, ph = 0;
            int s = 0;
            const uint32_t ring_addr = smem_u32(ring);
            // descriptor of a K-major 128-byte-swizzled operand at shared address 0: the address field is added per use
            const uint64_t desc0 = smem_desc(0, 16, 1024);
            for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++nacc) {
                const int buf = nacc & 1;
                if (nacc >= 2) PJ_WAIT(&acc_empty[buf], (nacc >> 1) - 1, 82);
                tc_fence_after();
                const uint32_t dcol = tmem_base + (uint32_t)(buf * BN);
                for (int i0 = 0; i0 < kb_count; i0 += KPER) {
                    const int nblk = min(KPER, kb_count - i0);
                    PJ_WAIT(&full[s], ph, 83);
                    tc_fence_after();
                    uint32_t aaddr = ring_addr + (uint32_t)s * (uint32_t)kStage;
#pragma unroll
                    for (int j = 0; j < KPER; ++j, aaddr += (uint32_t)kBlock) {
                        if (j >= nblk) break;
                        const uint64_t ad = desc_at(desc0, aaddr);
                        const uint64_t bd = desc_at(desc0, aaddr + (uint32_t)a.a_bytes);
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)  // 16 columns = 32 bytes = 2 units of the address field
                            umma_bf16(dcol, ad + 2 * kk, bd + 2 * kk, idesc, (i0 > 0) || (j > 0) || (kk > 0));
                    }
                    umma_commit(&empty[s]);
                    if (++s == a.stages) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
                umma_commit(&acc_full[buf]);
            }
        }
        __syncwarp();
    } else {
        // =========================== epilogue: one thread per output row ===========================
        const int quarter = warp & 3;  // the tensor-memory lanes this warp may read
        const int row = quarter * 32 + lane;
        uint32_t nacc = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++nacc) {
            int seg, n0, m0;
            locate(tile, &seg, &n0, &m0);
            const int buf = nacc & 1;
            PJ_WAIT(&acc_full[buf], nacc / 2, 84);
            tc_fence_after();
            const long long m = (long long)m0 + row;
            __nv_bfloat16* obase = seg == 0 ? a.out[0] : (seg == 1 ? a.out[1] : a.out[2]);
            const int n_feat = seg == 0 ? a.n_seg[0] : (seg == 1 ? a.n_seg[1] : a.n_seg[2]);
            __nv_bfloat16* dst = obase + (size_t)m * n_feat + n0;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN);
#pragma unroll
            for (int c = 0; c < BN / 32; ++c) {
                float y[32];
                tmem_ld32(taddr + c * 32, y);
                if (m < a.M && !*abort_flag) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        reinterpret_cast<uint4*>(dst + c * 32)[j] = Chunk<__nv_bfloat16>::pack(y + 8 * j);
                }
            }
            tc_fence_before();
            mbar_arrive(&acc_empty[buf]);
        }
    }
#undef PJ_WAIT

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// [rows][K] bfloat16, row-major, as a 2-D tensor (column, row); boxes of 64 columns x `box_rows` rows
// with the 128-byte swizzle; what lies outside reads as zeros.
bool make_matrix_map(CUtensorMap* map, const void* base, long long rows, int K, int box_rows) {
    if (box_rows > 256) return false;
    TensorMapEncodeFn fn = tensor_map_encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kPjBK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, int KPER>
cudaError_t launch_bn(const CUtensorMap& mx, const CUtensorMap& m0, const CUtensorMap& m1, const CUtensorMap& m2,
                      PjArgs a, int device, int sm_count, int smem_optin, cudaStream_t stream) {
    const int kStage = KPER * (a.a_bytes + BN * kPjBK * 2);
    const int pad = kPjABytes - a.a_bytes;  // the 128-row operand read of the last stage stays inside the allocation
    int stages = (smem_optin - 2048 - pad) / kStage;
    if (stages > kPjMaxStages) stages = kPjMaxStages;
    if (stages < 2) return cudaErrorInvalidConfiguration;
    a.stages = stages;
    const int smem = stages * kStage + pad + (2 * kPjMaxStages + 8) * 8 + 1024;
    auto fn = project_kernel<BN, KPER>;
    // the shared-memory limit of this kernel on this device is raised only when it has to grow (a decode
    // step's projection is short enough for one more runtime call per launch to show)
    static std::mutex smem_mu;
    static int smem_set[64] = {};
    std::lock_guard<std::mutex> smem_lock(smem_mu);
    if (device < 0 || device >= 64 || smem_set[device] < smem) {
        cudaError_t e = cudaFuncSetAttribute(reinterpret_cast<const void*>(fn), cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        if (device >= 0 && device < 64) smem_set[device] = smem;
    }
    const long long m_tiles = (a.M + kPjBM - 1) / kPjBM;
    const long long tiles = m_tiles * ((a.n_seg[0] + a.n_seg[1] + a.n_seg[2]) / BN);
    const int grid = (int)(tiles < sm_count ? tiles : sm_count);
    fn<<<grid, kPjThreads, smem, stream>>>(mx, m0, m1, m2, a);
    return cudaGetLastError();
}

}  // namespace

// q = x W_q^T, k = x W_wq^T, v = x W_wv^T for n_tokens rows of x.  Returns the CUDA error of the launch.
cudaError_t launch_project(long long n_tokens, int d_model, int n_q, int n_kv, const void* x, const void* w_q,
                           const void* w_wq, const void* w_wv, void* q, void* k, void* v, int* status, int device,
                           int sm_count, int smem_optin, cudaStream_t stream) {
    // feature tiles: 256 wide for long blocks of tokens (fewest operand bytes per product), 128 for
    // shorter ones, 64 (else 32) for a decode step (more tiles than SMs while the weights stream once)
    int BN = 32;
    if (n_q % 64 == 0 && n_kv % 64 == 0) BN = 64;
    const long long m_tiles = (n_tokens + kPjBM - 1) / kPjBM;
    // 128 wide when that still leaves about two thirds of the SMs a tile (a decode step of a model with
    // 12288 output features: 96 tiles on 148 SMs), or when there are several row tiles anyway
    if (n_q % 128 == 0 && n_kv % 128 == 0 && (n_tokens > 256 || m_tiles * ((n_q + 2 * n_kv) / 128) * 8 >= 5LL * sm_count))
        BN = 128;
    if (n_tokens >= 1024 && n_q % 256 == 0 && n_kv % 256 == 0) BN = 256;
    const int a_rows = n_tokens >= kPjBM ? kPjBM : (int)((n_tokens + 7) / 8 * 8);
    alignas(64) CUtensorMap mx, m0, m1, m2;
    if (!make_matrix_map(&mx, x, n_tokens, d_model, a_rows) || !make_matrix_map(&m0, w_q, n_q, d_model, BN) ||
        !make_matrix_map(&m1, w_wq, n_kv, d_model, BN) || !make_matrix_map(&m2, w_wv, n_kv, d_model, BN))
        return cudaErrorInvalidValue;
    PjArgs a;
    a.out[0] = static_cast<__nv_bfloat16*>(q);
    a.out[1] = static_cast<__nv_bfloat16*>(k);
    a.out[2] = static_cast<__nv_bfloat16*>(v);
    a.status = status;
    a.n_seg[0] = n_q;
    a.n_seg[1] = n_kv;
    a.n_seg[2] = n_kv;
    a.M = n_tokens;
    a.K = d_model;
    a.stages = 0;
    a.a_rows = a_rows;
    a.a_bytes = a_rows * kPjBK * 2;
    // Small blocks travel four or two to a stage while three stages still fit: measured at 64 tokens,
    // d_model 4096, 12288 features, every halving of the hand-overs per byte paid (64-wide tiles:
    // 57.6 / 43.1 / 34.8 us with 1 / 2 / 4 blocks per stage; 128-wide: 33.0 / 28.1 us with 1 / 2).
    const int block = a.a_bytes + BN * kPjBK * 2;
    int kper = 12 * block <= 200 * 1024 ? 4 : (6 * block <= 200 * 1024 ? 2 : 1);
#define PJ_LAUNCH(bn, kp) \
    if (BN == bn && kper == kp) return launch_bn<bn, kp>(mx, m0, m1, m2, a, device, sm_count, smem_optin, stream);
    PJ_LAUNCH(256, 1)
    PJ_LAUNCH(256, 2)
    PJ_LAUNCH(128, 1)
    PJ_LAUNCH(128, 2)
    PJ_LAUNCH(64, 1)
    PJ_LAUNCH(64, 2)
    PJ_LAUNCH(64, 4)
    PJ_LAUNCH(32, 1)
    PJ_LAUNCH(32, 2)
    PJ_LAUNCH(32, 4)
#undef PJ_LAUNCH
    return cudaErrorInvalidConfiguration;
}

}  // namespace bct
