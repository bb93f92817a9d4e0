// Partitioned causal GQA attention on tcgen05 tensor cores (bf16 operands, head_dim 128):
// the queries of one chunk against the key/value prefix that ends with the chunk.
//
// Forward, one CTA per (128-query tile, query head):
//   warp 0     : TMA producer -- Q once, then K and V tiles of 128 keys through two-stage rings
//   warp 1     : MMA issuer   -- S_j = Q K_j^T into one of two tensor-memory buffers (so S_{j+1} is
//                computed while the softmax of S_j runs), then O += P_j V_j
//   warps 2..5 : softmax      -- one query row per thread: row max and sum need no shuffles;
//                P_j is written to shared memory in the swizzled K-major layout the MMA reads;
//                the running output in tensor memory is rescaled only when a row's maximum
//                grows by more than 2^8 (exact: the final division by the row sum uses the same
//                reference), which after the first tiles is rare
//   Key tiles beyond the diagonal are never loaded; the causal predicate is evaluated only in
//   tiles the diagonal crosses.
//
// All mbarrier waits are bounded (see sm100.cuh); on expiry the CTA leaves its loops, frees its
// tensor memory and returns, and the host sees STREAMBP_E_DEVICE_TIMEOUT.
#include "sm100.cuh"

namespace sbp {
namespace {

constexpr int TILE = 128;                 // queries per CTA, keys per tile, head_dim
constexpr int HALF_BYTES = TILE * 64 * 2; // one [128 rows][64 cols] swizzled sub-tile
constexpr int TILE_BYTES = 2 * HALF_BYTES;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// A / B descriptors for a [128 rows][128 cols] bf16 tile stored as two 64-column swizzled sub-tiles.
// K-major use (contraction along the 128 columns): slice kk covers columns 16kk .. 16kk+15.
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t tile, int kk) {
    return make_desc_sw128(tile + (kk >> 2) * HALF_BYTES + (kk & 3) * 32, 16, 1024);
}
// MN-major use as B (contraction along the 128 rows, N = the 128 columns): slice kk covers rows 16kk .. 16kk+15.
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t tile, int kk) {
    return make_desc_sw128(tile + kk * 2048, HALF_BYTES, 1024);
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&h);
}
// 16-byte chunk `chunk` (0..15) of row `row` in a two-sub-tile swizzled [128][128] bf16 tile
__device__ __forceinline__ uint32_t swz_addr(uint32_t tile, int row, int chunk) {
    return tile + (chunk >> 3) * HALF_BYTES + row * 128 + (((chunk & 7) ^ (row & 7)) << 4);
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

struct FwdParams {
    int n;              // query rows in this chunk
    long long q0;       // absolute row of query 0
    int Hq, Hkv;
    bf16 *o;            // [n, Hq, 128]
    float *lse;         // [Hq, n]
    float scale_log2;   // log2(e) / sqrt(head_dim)
};

constexpr int FWD_SMEM = TILE_BYTES /*Q*/ + 2 * TILE_BYTES /*K*/ + 2 * TILE_BYTES /*V*/ + TILE_BYTES /*P*/ + 1024 + 256;

__global__ void __launch_bounds__(192, 1)
    attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                       const __grid_constant__ CUtensorMap map_v, const FwdParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const uint32_t sQ = base, sK = sQ + TILE_BYTES, sV = sK + 2 * TILE_BYTES, sP = sV + 2 * TILE_BYTES;
    uint8_t *aux = smem_raw + (base - raw) + 6 * TILE_BYTES;
    const uint32_t bars = smem_u32(aux);
    const uint32_t q_full = bars, k_full = bars + 8, k_empty = bars + 24, v_full = bars + 40, v_empty = bars + 56,
                   s_full = bars + 72, s_empty = bars + 88, p_full = bars + 104, pv_done = bars + 112;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(aux + 128);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(aux + 136);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = blockIdx.y, g = h / (p.Hq / p.Hkv);
    const int qt0 = blockIdx.x * TILE;
    const long long q_abs0 = p.q0 + qt0;                                      // absolute row of the tile's first query
    const int rows_here = (p.n - qt0) < TILE ? (p.n - qt0) : TILE;
    const long long kv_end = q_abs0 + rows_here;                              // keys 0 .. kv_end-1 are visible to the tile
    const int nkv = (int)((kv_end + TILE - 1) / TILE);

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < 2; s++) {
            mbar_init(k_full + 8 * s, 1);
            mbar_init(k_empty + 8 * s, 1);
            mbar_init(v_full + 8 * s, 1);
            mbar_init(v_empty + 8 * s, 1);
            mbar_init(s_full + 8 * s, 1);
            mbar_init(s_empty + 8 * s, 4);
        }
        mbar_init(p_full, 4);
        mbar_init(pv_done, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tS = tmem, tO = tmem + 256;     // S buffers at columns 0 and 128, O at 256

    if (warp == 0) {
        if (lane == 0) {
            mbar_expect_tx(q_full, TILE_BYTES);
            tma_load_2d(sQ, &map_q, q_full, h * TILE, qt0);
            tma_load_2d(sQ + HALF_BYTES, &map_q, q_full, h * TILE + 64, qt0);
            for (int j = 0; j < nkv; j++) {
                const uint32_t st = j & 1, ph = (j >> 1) & 1;
                if (!mbar_wait(k_empty + 8 * st, ph ^ 1u, abort_flag)) break;
                mbar_expect_tx(k_full + 8 * st, TILE_BYTES);
                tma_load_2d(sK + st * TILE_BYTES, &map_k, k_full + 8 * st, g * TILE, j * TILE);
                tma_load_2d(sK + st * TILE_BYTES + HALF_BYTES, &map_k, k_full + 8 * st, g * TILE + 64, j * TILE);
                if (!mbar_wait(v_empty + 8 * st, ph ^ 1u, abort_flag)) break;
                mbar_expect_tx(v_full + 8 * st, TILE_BYTES);
                tma_load_2d(sV + st * TILE_BYTES, &map_v, v_full + 8 * st, g * TILE, j * TILE);
                tma_load_2d(sV + st * TILE_BYTES + HALF_BYTES, &map_v, v_full + 8 * st, g * TILE + 64, j * TILE);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc_s = make_idesc(TILE, TILE, false, false);
            constexpr uint32_t idesc_pv = make_idesc(TILE, TILE, false, true);
            bool alive = mbar_wait(q_full, 0, abort_flag);
            auto issue_s = [&](int j) -> bool {
                const uint32_t st = j & 1, ph = (j >> 1) & 1;
                if (!mbar_wait(s_empty + 8 * st, ph ^ 1u, abort_flag)) return false;
                if (!mbar_wait(k_full + 8 * st, ph, abort_flag)) return false;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; kk++)
                    umma_bf16(tS + st * TILE, desc_kmajor(sQ, kk), desc_kmajor(sK + st * TILE_BYTES, kk), idesc_s,
                              kk != 0);
                umma_commit(k_empty + 8 * st);
                umma_commit(s_full + 8 * st);
                return true;
            };
            if (alive) alive = issue_s(0);
            for (int j = 0; j < nkv && alive; j++) {
                if (j + 1 < nkv && !issue_s(j + 1)) { alive = false; break; }
                const uint32_t st = j & 1, ph = (j >> 1) & 1;
                if (!mbar_wait(p_full, j & 1, abort_flag)) { alive = false; break; }
                if (!mbar_wait(v_full + 8 * st, ph, abort_flag)) { alive = false; break; }
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; kk++)
                    umma_bf16(tO, desc_kmajor(sP, kk), desc_mnmajor(sV + st * TILE_BYTES, kk), idesc_pv,
                              (j | kk) != 0);
                umma_commit(v_empty + 8 * st);
                umma_commit(pv_done);
            }
        }
    } else {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;                     // query row within the tile
        const long long q_abs = q_abs0 + row;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        float m_used = -INFINITY, l = 0.f;
        bool alive = true;
        for (int j = 0; j < nkv && alive; j++) {
            const uint32_t st = j & 1, ph = (j >> 1) & 1;
            if (!mbar_wait(s_full + 8 * st, ph, abort_flag)) { alive = false; break; }
            tc_fence_after();
            const uint32_t tSj = tS + st * TILE + lane_base;
            const long long k_abs0 = (long long)j * TILE;
            const bool diag = k_abs0 + TILE - 1 > q_abs0;       // some (query, key) pair of the tile is masked
            const int lim = diag ? (int)(q_abs - k_abs0) : (1 << 30);   // keys 0..lim of the tile are visible
            // pass 1: row maximum of the scaled scores
            float mt = -INFINITY;
#pragma unroll 1
            for (int c = 0; c < 4; c++) {
                uint32_t r[32];
                tmem_ld32(tSj + c * 32, r);
#pragma unroll
                for (int e = 0; e < 32; e++) {
                    float x = __uint_as_float(r[e]) * p.scale_log2;
                    if (c * 32 + e > lim) x = -INFINITY;
                    mt = fmaxf(mt, x);
                }
            }
            float factor = 1.f;
            const bool grow = mt > m_used + 8.f;                 // also true on the first tile (m_used = -inf)
            if (grow) {
                factor = fast_exp2(m_used - mt);
                m_used = mt;
                l *= factor;
            }
            // pass 2: P = exp2(x - m_used), packed to bf16
            uint32_t pk[64];
#pragma unroll
            for (int c = 0; c < 4; c++) {
                uint32_t r[32];
                tmem_ld32(tSj + c * 32, r);
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    float x0 = __uint_as_float(r[e]) * p.scale_log2 - m_used;
                    float x1 = __uint_as_float(r[e + 1]) * p.scale_log2 - m_used;
                    if (c * 32 + e > lim) x0 = -INFINITY;
                    if (c * 32 + e + 1 > lim) x1 = -INFINITY;
                    const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                    l += p0 + p1;
                    pk[c * 16 + e / 2] = pack_bf16(p0, p1);
                }
            }
            // S buffer may be overwritten by S_{j+2}
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(s_empty + 8 * st);
            // P buffer and O are free once P_{j-1} V_{j-1} has completed
            if (j > 0) {
                if (!mbar_wait(pv_done, (j - 1) & 1, abort_flag)) { alive = false; break; }
                tc_fence_after();
                if (__any_sync(0xffffffffu, grow)) {
#pragma unroll 1
                    for (int c = 0; c < 4; c++) {
                        uint32_t r[32];
                        tmem_ld32(tO + lane_base + c * 32, r);
#pragma unroll
                        for (int e = 0; e < 32; e++) r[e] = __float_as_uint(__uint_as_float(r[e]) * factor);
                        tmem_st32(tO + lane_base + c * 32, r);
                    }
                    tmem_wait_st();
                }
            }
#pragma unroll
            for (int cc = 0; cc < 16; cc++)
                st_shared_v4(swz_addr(sP, row, cc), pk[4 * cc], pk[4 * cc + 1], pk[4 * cc + 2], pk[4 * cc + 3]);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_full);
        }
        // epilogue: O / l and the log-sum-exp
        if (alive && mbar_wait(pv_done, (nkv - 1) & 1, abort_flag)) {
            tc_fence_after();
            const float inv = 1.f / l;
            const int qr = qt0 + row;
#pragma unroll 1
            for (int c = 0; c < 4; c++) {
                uint32_t r[32];
                tmem_ld32(tO + lane_base + c * 32, r);
                if (qr < p.n) {
                    bf16 *out = p.o + ((long long)qr * p.Hq + h) * TILE + c * 32;
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint32_t w[4];
#pragma unroll
                        for (int t = 0; t < 4; t++)
                            w[t] = pack_bf16(__uint_as_float(r[e + 2 * t]) * inv, __uint_as_float(r[e + 2 * t + 1]) * inv);
                        *reinterpret_cast<uint4 *>(out + e) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
            if (qr < p.n) p.lse[(long long)h * p.n + qr] = (m_used + log2f(l)) * kLn2;
        }
    }

    __syncwarp();
    if (*abort_flag) {
        const unsigned long long t0 = global_timer();
        while (global_timer() - t0 < 200000ull) { }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, 512);
    }
}

template <typename K>
bool opt_in_smem(K kernel, int bytes) {
    return cuda_ok(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
}

}  // namespace

bool attention_tc_supported(int64_t n, int64_t q0, int Hq, int Hkv, int dh, const void *q, const void *k,
                            const void *v) {
    if (dh != TILE || n < 1 || q0 < 0 || Hq % Hkv) return false;
    auto al = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
    if (!al(q) || !al(k) || !al(v)) return false;
    return tensor_maps_available();
}

int attention_fwd_tc(const bf16 *q, const bf16 *k, const bf16 *v, int64_t n, int64_t q0, int Hq, int Hkv, bf16 *o,
                     float *lse, cudaStream_t st) {
    CUtensorMap mq, mk, mv;
    const int64_t kv_len = q0 + n;
    if (!make_tensor_map(&mq, q, n, (int64_t)Hq * TILE, (int64_t)Hq * TILE, 64, TILE, false) ||
        !make_tensor_map(&mk, k, kv_len, (int64_t)Hkv * TILE, (int64_t)Hkv * TILE, 64, TILE, false) ||
        !make_tensor_map(&mv, v, kv_len, (int64_t)Hkv * TILE, (int64_t)Hkv * TILE, 64, TILE, false))
        return STREAMBP_E_CUDA;
    static bool configured = false;
    if (!configured) {
        if (!opt_in_smem(attn_fwd_tc_kernel, FWD_SMEM)) return STREAMBP_E_CUDA;
        configured = true;
    }
    FwdParams p{(int)n, (long long)q0, Hq, Hkv, o, lse, kLog2e / sqrtf((float)TILE)};
    dim3 grid((unsigned)((n + TILE - 1) / TILE), Hq);
    SBP_LAUNCH(attn_fwd_tc_kernel, grid, 192, FWD_SMEM, st, mq, mk, mv, p);
    return STREAMBP_OK;
}

int attention_tc_take_fault() { return take_fault_local(); }

}  // namespace sbp
