// tcgen05 tensor-core GEMM for sm_100a: bf16 operands staged in shared memory by TMA
// (128-byte swizzle), fp32 accumulation in tensor memory, three operand layouts.
//
//   persistent grid, one CTA per SM, output tile 128 x 256, K slices of 64
//   warp 0      : TMA producer (one elected lane)
//   warp 1      : allocates tensor memory, issues tcgen05.mma (one elected lane)
//   warps 2..5  : epilogue -- tcgen05.ld of a 32-lane quarter, bias, then
//                 fp32 output: 32x32 blocks staged in shared memory (128-byte swizzle) and written
//                 by TMA store, or added into C by TMA reduce-add when accumulating, so the
//                 read-modify-write of a weight-gradient tile never passes through the SM;
//                 bf16 output: 16-byte stores from registers
//   tensor memory holds two 128 x 256 fp32 accumulators, so the epilogue of tile i overlaps
//   the main loop of tile i+1.
//
// Operand layouts (GemmOp): K-major operands are loaded as [rows][64 k] boxes, MN-major operands
// (the B of "NN", both operands of "TN") as [64 k][64 mn] boxes; the shared-memory matrix
// descriptors tell the tensor core which of the two it is looking at, so no operand is ever
// transposed in memory.
//
// Every mbarrier wait is bounded (2 s of %globaltimer): on expiry the CTA raises a fault flag that
// streambp_last_device_status() reports as STREAMBP_E_DEVICE_TIMEOUT, all roles leave their loops,
// tensor memory is released and the kernel returns.
#include "sm100.cuh"

namespace sbp {
namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;   // 16 KiB
constexpr int B_BYTES = BN * BK * 2;   // 32 KiB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int EPI_BUF_BYTES = 32 * 128;                  // one 32 x 32 fp32 block
constexpr int EPI_BYTES = 4 * 2 * EPI_BUF_BYTES;          // 4 epilogue warps, double-buffered
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;
constexpr int NUM_THREADS = 192;
constexpr uint32_t TMEM_COLS = 512;

}  // namespace

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

namespace {
EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

}  // namespace

bool tensor_maps_available() { return encode_fn() != nullptr; }

// 2-D tensor map over a row-major [rows, cols] matrix with leading dimension ld (elements).
bool make_tensor_map(CUtensorMap *map, const void *base, int64_t rows, int64_t cols, int64_t ld, uint32_t box_cols,
                     uint32_t box_rows, bool f32) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * (f32 ? 4 : 2)};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(map, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        call_state().cuda_error = (int)r;
        return false;
    }
    return true;
}

int sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            n = 148;
    }
    return n;
}


namespace {

struct TcParams {
    int M, N, K;
    void *C;
    long long ldc;
    const bf16 *bias;
    int accumulate;
    const int *gate;      // optional: the kernel returns at once when *gate == 0
};

template <bool A_MN, bool B_MN, bool OUT_F32>
__global__ void __launch_bounds__(NUM_THREADS, 1)
    gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                   const __grid_constant__ CUtensorMap map_c, const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    if (gated_off(p.gate)) return;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;          // 1024-byte aligned operand stages
    const uint32_t epi = tiles + STAGES * STAGE_BYTES;      // fp32 staging blocks, 1024-byte aligned
    uint8_t *aux = smem_raw + (tiles - raw) + STAGES * STAGE_BYTES + EPI_BYTES;
    const uint32_t bar_full = smem_u32(aux);                 // STAGES x 8 B
    const uint32_t bar_empty = bar_full + 8 * STAGES;        // STAGES x 8 B
    const uint32_t bar_tfull = bar_empty + 8 * STAGES;       // 2 x 8 B
    const uint32_t bar_tempty = bar_tfull + 16;              // 2 x 8 B
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(aux + 8 * STAGES * 2 + 32);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(aux + 8 * STAGES * 2 + 40);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_m = (p.M + BM - 1) / BM, tiles_n = (p.N + BN - 1) / BN;
    const int num_tiles = tiles_m * tiles_n;
    const int num_kb = (p.K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; s++) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; b++) {
            mbar_init(bar_tfull + 8 * b, 1);
            mbar_init(bar_tempty + 8 * b, 4);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool alive = true;
            for (int tile = blockIdx.x; tile < num_tiles && alive; tile += gridDim.x) {
                const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
                for (int kb = 0; kb < num_kb; kb++) {
                    if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag)) { alive = false; break; }
                    const uint32_t full = bar_full + 8 * stage;
                    const uint32_t sa = tiles + stage * STAGE_BYTES, sb = sa + A_BYTES;
                    mbar_expect_tx(full, STAGE_BYTES);
                    const int k0 = kb * BK;
                    if (A_MN) {
#pragma unroll
                        for (int j = 0; j < BM / 64; j++) tma_load_2d(sa + j * 8192, &map_a, full, m0 + 64 * j, k0);
                    } else {
                        tma_load_2d(sa, &map_a, full, k0, m0);
                    }
                    if (B_MN) {
#pragma unroll
                        for (int j = 0; j < BN / 64; j++) tma_load_2d(sb + j * 8192, &map_b, full, n0 + 64 * j, k0);
                    } else {
                        tma_load_2d(sb, &map_b, full, k0, n0);
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) |
                                       ((B_MN ? 1u : 0u) << 16) | ((uint32_t)(BN >> 3) << 17) |
                                       ((uint32_t)(BM >> 4) << 24);
            constexpr uint32_t a_step = A_MN ? 2048u : 32u, b_step = B_MN ? 2048u : 32u;  // bytes per 16 k
            uint32_t stage = 0, phase = 0, local = 0;
            bool alive = true;
            for (int tile = blockIdx.x; tile < num_tiles && alive; tile += gridDim.x, local++) {
                const uint32_t buf = local & 1u, use = local >> 1;
                if (!mbar_wait(bar_tempty + 8 * buf, (use & 1u) ^ 1u, abort_flag)) { alive = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0; kb < num_kb; kb++) {
                    if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag)) { alive = false; break; }
                    tc_fence_after();
                    const uint32_t sa = tiles + stage * STAGE_BYTES, sb = sa + A_BYTES;
                    const uint32_t a_lo = desc_lo(sa, A_MN ? 8192u : 16u), b_lo = desc_lo(sb, B_MN ? 8192u : 16u);
#pragma unroll
                    for (int kk = 0; kk < BK / 16; kk++)
                        umma_ss(d_tmem, a_lo + kk * (a_step >> 4), b_lo + kk * (b_step >> 4), idesc,
                                (kb | kk) != 0 ? 1u : 0u);
                    umma_commit(bar_empty + 8 * stage);   // frees the stage once these MMAs have read it
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (alive) umma_commit(bar_tfull + 8 * buf);   // accumulator complete
            }
        }
    } else {
        // ------------------------------ epilogue ------------------------------
        const int quarter = warp & 3;                 // TMEM lanes 32*quarter .. +31
        uint32_t local = 0, staged = 0;               // staged: fp32 blocks this warp has sent so far
        bool alive = true;
        for (int tile = blockIdx.x; tile < num_tiles && alive; tile += gridDim.x, local++) {
            const int m0 = (tile % tiles_m) * BM, n0 = (tile / tiles_m) * BN;
            const uint32_t buf = local & 1u, use = local >> 1;
            if (!mbar_wait(bar_tfull + 8 * buf, use & 1u, abort_flag)) { alive = false; break; }
            tc_fence_after();
            const int row = m0 + quarter * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * BN;
#pragma unroll 1
            for (int c = 0; c < BN / 32; c++) {
                const int col0 = n0 + c * 32;
                if (col0 >= p.N) break;               // uniform across the warp
                uint32_t r[32];
                tmem_ld32(taddr + c * 32, r);
                if (OUT_F32) {
                    // stage the warp's 32 x 32 block (row = lane) with the 128-byte swizzle the tensor map expects
                    const uint32_t buf_s = epi + (uint32_t)(quarter * 2 + (staged & 1u)) * EPI_BUF_BYTES;
                    staged++;
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 8; j++) {
                        float v[4];
#pragma unroll
                        for (int e = 0; e < 4; e++) {
                            v[e] = __uint_as_float(r[4 * j + e]);
                            if (p.bias && col0 + 4 * j + e < p.N) v[e] += __bfloat162float(p.bias[col0 + 4 * j + e]);
                        }
                        const uint32_t dst = buf_s + lane * 128 + ((j ^ (lane & 7)) << 4);
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(v[0]), "f"(v[1]),
                                     "f"(v[2]), "f"(v[3])
                                     : "memory");
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        if (p.accumulate) tma_reduce_add_2d(&map_c, buf_s, col0, m0 + quarter * 32);
                        else tma_store_2d(&map_c, buf_s, col0, m0 + quarter * 32);
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                } else if (row < p.M) {
                    {
                        bf16 *out = reinterpret_cast<bf16 *>(p.C) + (long long)row * p.ldc + col0;
#pragma unroll
                        for (int j = 0; j < 32; j += 8) {
                            float v[8];
#pragma unroll
                            for (int e = 0; e < 8; e++) {
                                v[e] = __uint_as_float(r[j + e]);
                                if (p.bias && col0 + j + e < p.N) v[e] += __bfloat162float(p.bias[col0 + j + e]);
                            }
                            if (col0 + j + 7 < p.N) {
                                uint32_t w[4];
#pragma unroll
                                for (int e = 0; e < 4; e++) {
                                    __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
                                    w[e] = *reinterpret_cast<uint32_t *>(&h);
                                }
                                *reinterpret_cast<uint4 *>(out + j) = make_uint4(w[0], w[1], w[2], w[3]);
                            } else {
                                for (int e = 0; e < 8; e++)
                                    if (col0 + j + e < p.N) out[j + e] = __float2bfloat16_rn(v[e]);
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
        }
    }

    if (OUT_F32 && warp >= 2 && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    __syncwarp();
    if (*abort_flag) {
        // give copies that are still in flight time to land before shared memory is released
        const unsigned long long t0 = global_timer();
        while (global_timer() - t0 < 200000ull) { }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
template <bool A_MN, bool B_MN, bool OUT_F32>
int launch(const CUtensorMap &ma, const CUtensorMap &mb, const CUtensorMap &mc, const TcParams &p, cudaStream_t st) {
    auto kernel = gemm_tc_kernel<A_MN, B_MN, OUT_F32>;
    static bool configured = false;
    if (!configured) {
        if (!cuda_ok(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES)))
            return STREAMBP_E_CUDA;
        configured = true;
    }
    const int tiles = ((p.M + BM - 1) / BM) * ((p.N + BN - 1) / BN);
    const int grid = tiles < sm_count() ? tiles : sm_count();
    SBP_LAUNCH(kernel, grid, NUM_THREADS, SMEM_BYTES, st, ma, mb, mc, p);
    return STREAMBP_OK;
}

}  // namespace

bool gemm_tc_supported(GemmOp op, int64_t M, int64_t N, int64_t K, int64_t lda, int64_t ldb, int64_t ldc,
                       const void *A, const void *B, const void *C, bool c_is_f32) {
    (void)op;
    if (M < 1 || N < 1 || K < 1 || M > (1ll << 30) || N > (1ll << 30) || K > (1ll << 30)) return false;
    if ((lda % 8) || (ldb % 8)) return false;                       // TMA: 16-byte row pitch
    if (ldc % (c_is_f32 ? 4 : 8)) return false;                     // 16-byte vector stores
    auto al = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
    if (!al(A) || !al(B) || !al(C)) return false;
    return tensor_maps_available();
}

int gemm_tc(GemmOp op, int64_t M, int64_t N, int64_t K, const bf16 *A, int64_t lda, const bf16 *B, int64_t ldb,
            void *C, int64_t ldc, bool c_is_f32, const bf16 *bias, bool accumulate, cudaStream_t st) {
    CUtensorMap ma, mb;
    bool ok = true;
    switch (op) {
        case OP_NT:   // A [M,K] K-major, B [N,K] K-major
            ok = make_tensor_map(&ma, A, M, K, lda, BK, BM, false) && make_tensor_map(&mb, B, N, K, ldb, BK, BN, false);
            break;
        case OP_NN:   // A [M,K] K-major, B [K,N] N-major
            ok = make_tensor_map(&ma, A, M, K, lda, BK, BM, false) && make_tensor_map(&mb, B, K, N, ldb, 64, BK, false);
            break;
        case OP_TN:   // A [K,M] M-major, B [K,N] N-major
            ok = make_tensor_map(&ma, A, K, M, lda, 64, BK, false) && make_tensor_map(&mb, B, K, N, ldb, 64, BK, false);
            break;
    }
    CUtensorMap mc = ma;   // unused by the bf16-output kernels
    if (ok && c_is_f32) ok = make_tensor_map(&mc, C, M, N, ldc, 32, 32, true);
    if (!ok) return STREAMBP_E_CUDA;
    TcParams p{(int)M, (int)N, (int)K, C, (long long)ldc, bias, accumulate ? 1 : 0, call_state().gate};
    if (op == OP_NT) return c_is_f32 ? launch<false, false, true>(ma, mb, mc, p, st) : launch<false, false, false>(ma, mb, mc, p, st);
    if (op == OP_NN) return c_is_f32 ? launch<false, true, true>(ma, mb, mc, p, st) : launch<false, true, false>(ma, mb, mc, p, st);
    return c_is_f32 ? launch<true, true, true>(ma, mb, mc, p, st) : launch<true, true, false>(ma, mb, mc, p, st);
}

int gemm_tc_take_fault() { return take_fault_local(); }

}  // namespace sbp
