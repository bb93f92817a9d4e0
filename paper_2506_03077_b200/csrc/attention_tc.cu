// Partitioned causal GQA attention on tcgen05 tensor cores (bf16 operands, head_dim 128):
// the queries of one chunk against the key/value prefix that ends with the chunk.
//
// Forward, two kernels (attn_fwd_2q_kernel for chunks of more than 128 rows, attn_fwd_tc16_kernel otherwise):
//   warp 0      : TMA producer -- Q once, then K and V tiles of 128 keys through two-stage rings
//   warp 1      : MMA issuer   -- S_j = Q K_j^T into tensor memory, then O += P_j V_j with P_j read from
//                 tensor memory as the A operand
//   other warps : softmax      -- row maxima, exponentials, row sums, P packed to bf16 back into tensor
//                 memory; the running output in tensor memory is rescaled only when a row's maximum
//                 grows by more than 2^8 (exact: the final division by the row sum uses the same
//                 reference), which after the first tiles is rare
//   Key tiles beyond the diagonal are never loaded; the causal predicate is evaluated only in
//   tiles the diagonal crosses.  The two kernels differ in how the softmax work is laid out (see each).
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

// Descriptor low words for a [128 rows][128 cols] bf16 tile stored as two 64-column swizzled sub-tiles.
// K-major use (contraction along the 128 columns): slice kk covers columns 16kk .. 16kk+15.
__device__ __forceinline__ uint32_t klo(uint32_t tile) { return desc_lo(tile, 16); }
__host__ __device__ constexpr uint32_t kstep(int kk) { return (uint32_t)((kk >> 2) * (HALF_BYTES >> 4) + (kk & 3) * 2); }
// MN-major use as B (contraction along the 128 rows, N = the 128 columns): slice kk covers rows 16kk .. 16kk+15.
__device__ __forceinline__ uint32_t mnlo(uint32_t tile) { return desc_lo(tile, HALF_BYTES); }
__host__ __device__ constexpr uint32_t mnstep(int kk) { return (uint32_t)(kk * 128); }

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&h);
}
struct FwdParams {
    int n;              // query rows in this chunk
    long long q0;       // absolute row of query 0
    int Hq, Hkv;
    bf16 *o;            // [n, Hq, 128]
    float *lse;         // [Hq, n]
    float scale_log2;   // log2(e) / sqrt(head_dim)
};

// ---------------------------------------------------------------------------------------------
// Forward with sixteen softmax warps: the 128 key columns of a tile are split over four warpgroups
// (32 columns per thread), so four warps per scheduler hide the tensor-memory load latency that one
// warp per scheduler leaves exposed.  The four threads that share a query row exchange their partial
// row maxima through shared memory (an mbarrier with a bounded wait, not bar.sync, so that a CTA that
// is giving up cannot dead-lock on it); they then take identical rescale decisions, keep partial row
// sums that are only combined in the epilogue, and each warpgroup rescales / writes its own 32 head
// dims of the output.
// ---------------------------------------------------------------------------------------------
constexpr int FWD16_THREADS = 64 + 512;
constexpr int FWD16_SMEM = 5 * TILE_BYTES + 3 * 4 * TILE * 4 /* row max x2, row sum */ + 1024 + 256;

__global__ void __launch_bounds__(FWD16_THREADS, 1)
    attn_fwd_tc16_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                         const __grid_constant__ CUtensorMap map_v, const FwdParams p) {
    pdl_enter();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const uint32_t sQ = base, sK = sQ + TILE_BYTES, sV = sK + 2 * TILE_BYTES;
    uint8_t *tail = smem_raw + (base - raw) + 5 * TILE_BYTES;
    float *s_max = reinterpret_cast<float *>(tail);            // [2 buffers][4 groups][128 rows]
    float *s_sum = s_max + 2 * 4 * TILE;                       // [4 groups][128 rows]
    uint8_t *aux = tail + 3 * 4 * TILE * 4;
    const uint32_t bars = smem_u32(aux);
    const uint32_t q_full = bars, k_full = bars + 8, k_empty = bars + 24, v_full = bars + 40, v_empty = bars + 56,
                   s_full = bars + 72, s_empty = bars + 88, p_full = bars + 104, pv_done = bars + 112,
                   mx_bar = bars + 120, sum_bar = bars + 136;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(aux + 144);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(aux + 152);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // grid (heads, query tiles): the tiles with the longest key prefix are dispatched first
    const int h = blockIdx.x, g = h / (p.Hq / p.Hkv);
    const int qt0 = (int)(gridDim.y - 1 - blockIdx.y) * TILE;
    const long long q_abs0 = p.q0 + qt0;
    const int rows_here = (p.n - qt0) < TILE ? (p.n - qt0) : TILE;
    const long long kv_end = q_abs0 + rows_here;
    const int nkv = (int)((kv_end + TILE - 1) / TILE);

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < 2; s++) {
            mbar_init(k_full + 8 * s, 1);
            mbar_init(k_empty + 8 * s, 1);
            mbar_init(v_full + 8 * s, 1);
            mbar_init(v_empty + 8 * s, 1);
            mbar_init(s_full + 8 * s, 1);
            mbar_init(s_empty + 8 * s, 16);
            mbar_init(mx_bar + 8 * s, 16);
        }
        mbar_init(p_full, 16);
        mbar_init(pv_done, 1);
        mbar_init(sum_bar, 16);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tS = tmem, tO = tmem + 256, tP = tmem + 384;   // S x2, O, packed P (64 columns)

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
        // softmax-bound kernel: a single issuing lane leaves the other warps more issue slots
        if (lane == 0) {
            constexpr uint32_t idesc_s = make_idesc(TILE, TILE, false, false);
            constexpr uint32_t idesc_pv = make_idesc(TILE, TILE, false, true);
            bool alive = mbar_wait(q_full, 0, abort_flag);
            const uint32_t q_lo = klo(sQ);
            auto issue_s = [&](int j) -> bool {
                const uint32_t st = j & 1, ph = (j >> 1) & 1;
                if (!mbar_wait(s_empty + 8 * st, ph ^ 1u, abort_flag)) return false;
                if (!mbar_wait(k_full + 8 * st, ph, abort_flag)) return false;
                tc_fence_after();
                const uint32_t k_lo = klo(sK + st * TILE_BYTES);
#pragma unroll
                for (int kk = 0; kk < 8; kk++) umma_ss(tS + st * TILE, q_lo + kstep(kk), k_lo + kstep(kk), idesc_s, kk != 0);
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
                const uint32_t v_lo = mnlo(sV + st * TILE_BYTES);
#pragma unroll
                for (int kk = 0; kk < 8; kk++) umma_ts(tO, tP + kk * 8, v_lo + mnstep(kk), idesc_pv, (j | kk) != 0);
                umma_commit(v_empty + 8 * st);
                umma_commit(pv_done);
            }
        }
    } else {
        const int quarter = warp & 3;
        const int wg = (warp - 2) >> 2;                          // key-column group 0..3 (and head-dim group in O)
        const int col_base = wg * 32;
        const int row = quarter * 32 + lane;
        const long long q_abs = q_abs0 + row;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        float m_used = -INFINITY, l = 0.f;                       // l: partial row sum over this thread's columns
        bool alive = true;
        for (int j = 0; j < nkv && alive; j++) {
            const uint32_t st = j & 1, ph = (j >> 1) & 1;
            if (!mbar_wait(s_full + 8 * st, ph, abort_flag)) { alive = false; break; }
            tc_fence_after();
            const long long k_abs0 = (long long)j * TILE;
            const bool diag = k_abs0 + TILE - 1 > q_abs0;
            const int lim = (int)(q_abs - k_abs0);                // keys 0..lim of the tile are visible (diag tiles)
            uint32_t r[32];
            tmem_ld32(tS + st * TILE + col_base + lane_base, r);
            // S buffer may be overwritten by S_{j+2}
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(s_empty + 8 * st);
            float mt = -INFINITY;
            if (diag) {
#pragma unroll
                for (int e = 0; e < 32; e++) {
                    if (col_base + e > lim) r[e] = 0xff800000u;   // -inf
                    mt = fmaxf(mt, __uint_as_float(r[e]));
                }
            } else {
#pragma unroll
                for (int e = 0; e < 32; e++) mt = fmaxf(mt, __uint_as_float(r[e]));
            }
            // exchange partial maxima with the three other threads of this row
            s_max[(st * 4 + wg) * TILE + row] = mt;
            __syncwarp();
            if (lane == 0) mbar_arrive(mx_bar + 8 * st);
            if (!mbar_wait(mx_bar + 8 * st, ph, abort_flag)) { alive = false; break; }
            const float *mx = s_max + st * 4 * TILE + row;
            mt = fmaxf(fmaxf(mx[0], mx[TILE]), fmaxf(mx[2 * TILE], mx[3 * TILE])) * p.scale_log2;
            float factor = 1.f;
            const bool grow = mt > m_used + 8.f;                  // also true on the first tile (m_used = -inf)
            if (grow) {
                factor = fast_exp2(m_used - mt);
                m_used = mt;
                l *= factor;
            }
            uint32_t pk[16];
            const float neg_m = -m_used;
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
                const float p0 = fast_exp2(fmaf(__uint_as_float(r[e]), p.scale_log2, neg_m));
                const float p1 = fast_exp2(fmaf(__uint_as_float(r[e + 1]), p.scale_log2, neg_m));
                l += p0 + p1;
                pk[e / 2] = pack_bf16(p0, p1);
            }
            // P buffer and O are free once P_{j-1} V_{j-1} has completed
            if (j > 0) {
                if (!mbar_wait(pv_done, (j - 1) & 1, abort_flag)) { alive = false; break; }
                tc_fence_after();
                if (__any_sync(0xffffffffu, grow)) {              // this warpgroup rescales head dims col_base .. +31
                    uint32_t o[32];
                    tmem_ld32(tO + lane_base + col_base, o);
#pragma unroll
                    for (int e = 0; e < 32; e++) o[e] = __float_as_uint(__uint_as_float(o[e]) * factor);
                    tmem_st32(tO + lane_base + col_base, o);
                }
            }
            tmem_st16(tP + lane_base + wg * 16, pk);
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_full);
        }
        // epilogue: combine the four partial row sums, then O / l and the log-sum-exp
        if (alive) {
            s_sum[wg * TILE + row] = l;
            __syncwarp();
            if (lane == 0) mbar_arrive(sum_bar);
            if (mbar_wait(sum_bar, 0, abort_flag) && mbar_wait(pv_done, (nkv - 1) & 1, abort_flag)) {
                tc_fence_after();
                const float lt = s_sum[row] + s_sum[TILE + row] + s_sum[2 * TILE + row] + s_sum[3 * TILE + row];
                const float inv = 1.f / lt;
                const int qr = qt0 + row;
                uint32_t o[32];
                tmem_ld32(tO + lane_base + col_base, o);
                if (qr < p.n) {
                    bf16 *out = p.o + ((long long)qr * p.Hq + h) * TILE + col_base;
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint32_t w[4];
#pragma unroll
                        for (int t = 0; t < 4; t++)
                            w[t] = pack_bf16(__uint_as_float(o[e + 2 * t]) * inv, __uint_as_float(o[e + 2 * t + 1]) * inv);
                        *reinterpret_cast<uint4 *>(out + e) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                    if (wg == 0) p.lse[(long long)h * p.n + qr] = (m_used + log2f(lt)) * kLn2;
                }
            }
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

// ---------------------------------------------------------------------------------------------
// Forward with two query tiles per CTA.  The single-tile kernel above spends ~1100 of the ~2300 cycles of a
// key tile in latencies its sixteen softmax warps all sit through together (tensor-memory load, exchange of
// partial row maxima, store of P, barrier hand-offs), with the exp2 unit idle.  Here a CTA owns two adjacent
// 128-query tiles of one head, each with its own S / P and O in tensor memory and its own team of four softmax
// warps; the two teams are independent of each other, so one team's latencies fall into the other's
// exponential phase, and each K / V tile is fetched once for 256 query rows.
//   warp 0     : TMA producer -- both Q tiles once, then K and V tiles through two-stage rings
//   warp 1     : MMA issuer (warp-uniform issue) -- per key tile j and team X: S_X = Q_X K_j^T when the team has
//                finished with its previous P (P is packed into the columns of S, so the product that reads P is
//                queued before the one that overwrites S: the tensor pipe executes one thread's MMAs in order),
//                O_X += P_X V_j when the team has stored P_X
//   warps 2..9 : softmax, team (warp - 2) / 4 -- a thread owns a whole query row: 128 scores in registers, no
//                exchange between threads, row maximum and row sum private; lazy exact rescale as above
// ---------------------------------------------------------------------------------------------
constexpr int FWD2Q_THREADS = 64 + 256;
constexpr int FWD2Q_SMEM = 6 * TILE_BYTES + 1024 + 256;

__global__ void __launch_bounds__(FWD2Q_THREADS, 1)
    attn_fwd_2q_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                       const __grid_constant__ CUtensorMap map_v, const FwdParams p) {
    pdl_enter();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const uint32_t sQ = base, sK = sQ + 2 * TILE_BYTES, sV = sK + 2 * TILE_BYTES;
    uint8_t *aux = smem_raw + (base - raw) + 6 * TILE_BYTES;
    const uint32_t bars = smem_u32(aux);
    const uint32_t q_full = bars, k_full = bars + 8, k_empty = bars + 24, v_full = bars + 40, v_empty = bars + 56,
                   s_full = bars + 72, p_full = bars + 88, o_done = bars + 104;   // the last three: one per team
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(aux + 120);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(aux + 128);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // grid (heads, query tile pairs): the pairs with the longest key prefix are dispatched first
    const int h = blockIdx.x, g = h / (p.Hq / p.Hkv);
    const int qt0 = (int)(gridDim.y - 1 - blockIdx.y) * 2 * TILE;
    // team X: query rows qt0 + X * TILE .. ; its key tiles 0 .. nkv[X] - 1 (0 tiles: team absent)
    int nkv[2];
#pragma unroll
    for (int x = 0; x < 2; x++) {
        const int first = qt0 + x * TILE;
        const int rows = (p.n - first) < TILE ? (p.n - first) : TILE;
        nkv[x] = rows > 0 ? (int)((p.q0 + first + rows + TILE - 1) / TILE) : 0;
    }
    const int nkv_all = nkv[1] > nkv[0] ? nkv[1] : nkv[0];

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < 2; s++) {
            mbar_init(k_full + 8 * s, 1);
            mbar_init(k_empty + 8 * s, 1);
            mbar_init(v_full + 8 * s, 1);
            mbar_init(v_empty + 8 * s, 1);
            mbar_init(s_full + 8 * s, 1);
            mbar_init(p_full + 8 * s, 4);
            mbar_init(o_done + 8 * s, 1);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;      // columns: S_A 0..127, S_B 128..255, O_A 256..383, O_B 384..511

    if (warp == 0) {
        if (lane == 0) {
            mbar_expect_tx(q_full, (nkv[1] > 0 ? 2 : 1) * TILE_BYTES);
            for (int x = 0; x < 2; x++) {
                if (nkv[x] == 0) continue;
                tma_load_2d(sQ + x * TILE_BYTES, &map_q, q_full, h * TILE, qt0 + x * TILE);
                tma_load_2d(sQ + x * TILE_BYTES + HALF_BYTES, &map_q, q_full, h * TILE + 64, qt0 + x * TILE);
            }
            for (int j = 0; j < nkv_all; j++) {
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
        constexpr uint32_t idesc_s = make_idesc(TILE, TILE, false, false);
        constexpr uint32_t idesc_pv = make_idesc(TILE, TILE, false, true);
        bool alive = mbar_wait_warp(q_full, 0, abort_flag);
        auto issue_s = [&](int x, int j) {          // S_x = Q_x K_j^T (K_j is in shared memory)
            const uint32_t q_lo = klo(sQ + x * TILE_BYTES), k_lo = klo(sK + (j & 1) * TILE_BYTES);
#pragma unroll
            for (int kk = 0; kk < 8; kk++) umma_ss_w(tmem + x * TILE, q_lo + kstep(kk), k_lo + kstep(kk), idesc_s, kk != 0);
            umma_commit_w(s_full + 8 * x);
        };
        auto issue_pv = [&](int x, int j) -> bool {  // O_x += P_x V_j once the team has stored P_x
            if (!mbar_wait_warp(p_full + 8 * x, j & 1, abort_flag)) return false;
            tc_fence_after();
            const uint32_t v_lo = mnlo(sV + (j & 1) * TILE_BYTES);
#pragma unroll
            for (int kk = 0; kk < 8; kk++)
                umma_ts_w(tmem + 256 + x * TILE, tmem + x * TILE + kk * 8, v_lo + mnstep(kk), idesc_pv, (j | kk) != 0);
            if (j == nkv[x] - 1) umma_commit_w(o_done + 8 * x);
            return true;
        };
        if (alive) alive = mbar_wait_warp(k_full, 0, abort_flag);
        if (alive) {
            tc_fence_after();
            for (int x = 0; x < 2; x++)
                if (nkv[x] > 0) issue_s(x, 0);
            umma_commit_w(k_empty);
        }
        for (int j = 0; j < nkv_all && alive; j++) {
            const uint32_t st = j & 1, ph = (j >> 1) & 1;
            if (!mbar_wait_warp(v_full + 8 * st, ph, abort_flag)) { alive = false; break; }
            if (j + 1 < nkv_all && !mbar_wait_warp(k_full + 8 * ((j + 1) & 1), ((j + 1) >> 1) & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
            for (int x = 0; x < 2 && alive; x++) {
                if (j < nkv[x]) alive = issue_pv(x, j);
                if (alive && j + 1 < nkv[x]) issue_s(x, j + 1);
            }
            if (!alive) break;
            umma_commit_w(v_empty + 8 * st);
            if (j + 1 < nkv_all) umma_commit_w(k_empty + 8 * ((j + 1) & 1));
        }
    } else {
        const int x = (warp - 2) >> 2;                           // team
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const int first = qt0 + x * TILE;
        const long long q_abs0 = p.q0 + first, q_abs = q_abs0 + row;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        const uint32_t tS = tmem + x * TILE + lane_base, tO = tmem + 256 + x * TILE + lane_base;
        float m_used = -INFINITY, l = 0.f;
        bool alive = true;
        for (int j = 0; j < nkv[x] && alive; j++) {
            if (!mbar_wait(s_full + 8 * x, j & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
            uint32_t r[128];
#pragma unroll
            for (int c = 0; c < 4; c++) tmem_ld32_async(tS + c * 32, r + c * 32);
            tmem_wait_ld();
            const long long k_abs0 = (long long)j * TILE;
            if (k_abs0 + TILE - 1 > q_abs0) {                    // the diagonal crosses this tile
                const int lim = (int)(q_abs - k_abs0);            // keys 0..lim of the tile are visible
#pragma unroll
                for (int e = 0; e < 128; e++)
                    if (e > lim) r[e] = 0xff800000u;              // -inf
            }
            float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int e = 0; e < 128; e += 4) {
#pragma unroll
                for (int t = 0; t < 4; t++) m4[t] = fmaxf(m4[t], __uint_as_float(r[e + t]));
            }
            const float mt = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])) * p.scale_log2;
            float factor = 1.f;
            const bool grow = mt > m_used + 8.f;                  // also true on the first tile (m_used = -inf)
            if (grow) {
                factor = fast_exp2(m_used - mt);
                m_used = mt;
                l *= factor;
            }
            // S_j complete implies P_{j-1} V_{j-1} complete (same issuing thread, earlier in its order): O is at rest
            if (j > 0 && __any_sync(0xffffffffu, grow)) {
#pragma unroll 1
                for (int c = 0; c < 4; c++) {
                    uint32_t o[32];
                    tmem_ld32(tO + c * 32, o);
#pragma unroll
                    for (int e = 0; e < 32; e++) o[e] = __float_as_uint(__uint_as_float(o[e]) * factor);
                    tmem_st32(tO + c * 32, o);
                }
            }
            const float neg_m = -m_used;
            float l4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int c = 0; c < 8; c++) {                        // 16 scores -> 8 packed words per step
                uint32_t pk[8];
#pragma unroll
                for (int e = 0; e < 16; e += 2) {
                    const float p0 = fast_exp2(fmaf(__uint_as_float(r[c * 16 + e]), p.scale_log2, neg_m));
                    const float p1 = fast_exp2(fmaf(__uint_as_float(r[c * 16 + e + 1]), p.scale_log2, neg_m));
                    l4[(e >> 1) & 3] += p0 + p1;
                    pk[e >> 1] = pack_bf16(p0, p1);
                }
#pragma unroll
                for (int e = 0; e < 8; e++) r[c * 8 + e] = pk[e];  // packed P reuses the registers of consumed scores
            }
            l += (l4[0] + l4[1]) + (l4[2] + l4[3]);
            // P overwrites the first 64 columns of S (this thread's own lane)
#pragma unroll
            for (int c = 0; c < 4; c++) {
                uint32_t w[16];
#pragma unroll
                for (int e = 0; e < 16; e++) w[e] = r[c * 16 + e];
                tmem_st16(tS + c * 16, w);
            }
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_full + 8 * x);
        }
        if (alive && nkv[x] > 0 && mbar_wait(o_done + 8 * x, 0, abort_flag)) {
            tc_fence_after();
            const float inv = 1.f / l;
            const int qr = first + row;
#pragma unroll 1
            for (int c = 0; c < 4; c++) {
                uint32_t o[32];
                tmem_ld32(tO + c * 32, o);
                if (qr < p.n) {
                    bf16 *out = p.o + ((long long)qr * p.Hq + h) * TILE + c * 32;
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint32_t w[4];
#pragma unroll
                        for (int t = 0; t < 4; t++)
                            w[t] = pack_bf16(__uint_as_float(o[e + 2 * t]) * inv, __uint_as_float(o[e + 2 * t + 1]) * inv);
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

// ---------------------------------------------------------------------------------------------
// Backward.  Two CTA roles in one grid (attn_bwd_tc_kernel), both deterministic (no floating-point atomics):
//   dK/dV: one CTA per (128-key tile, KV head); K and V tiles stay in shared memory; loops over the
//          G query heads of the group and over the query tiles that can see the key tile.
//          S^T = K Q^T and dP^T = V dO^T land in tensor memory with keys on the lanes, so a thread owns
//          one key row.  The softmax warps read S^T and dP^T into registers and write BOTH packed bf16
//          operands -- P^T and dS^T -- over the columns of dP^T (first / second 16 columns of each 32-column
//          group), from where they feed dV += P^T dO and dK += dS^T Q as tensor-memory A operands.  The
//          columns of S^T are therefore free as soon as they have been read, and S^T of the next iteration is
//          queued at once, a whole iteration ahead (the Q ring has three stages for that: Q_i is read by
//          S^T_i and again, an iteration later, by dK_i); dP^T of the next iteration follows dK in the same
//          thread's issue order.  The Q / dO tiles serve both as K-major B operands (first two products) and
//          as MN-major B operands (last two) without being moved.
//   dQ   : one CTA per (128-query tile, query head); Q and dO tiles stay resident, K / V tiles stream;
//          S = Q K^T, dP = dO V^T, dS packed in place, dQ += dS K.
// Work inside a tile pair is split in TIME, not in space, so every product is a full 128 x 128 x 128 one
// (an N = 64 product is limited by shared-memory bandwidth to 2/3 of the tensor rate): the softmax
// warps (16 per CTA, each thread owns 32 columns of one row) first turn S into P -- which is all the dV
// product needs -- and only then combine it with dP into dS.
// Tensor memory is full in both roles (four 128-column fp32 tiles), which leaves one dependency cycle per
// iteration that cannot be cut: packed operands -> dK -> next dP^T -> softmax.  Timelines (clock64 stamps in
// the kernel) put an iteration of the dK/dV role at ~3000 cycles for 2048 cycles of products.  More overlap
// does not buy time on this part, though: run back to back for seconds, every variant of this kernel that was
// built -- a second issuing warp, Q / dO of the dQ role as tensor-memory operands, the older S^T-in-place
// scheme -- draws the board's full power limit and the clock settles so that the time per call is the same
// within 1-2 % (fewer cycles per tile, lower clock).  At the limit the kernel is bound by energy per tile
// pair, of which the seven products (five algorithmic + S and dP recomputed by the dQ role, the price of a
// deterministic result) are the bulk.
// ---------------------------------------------------------------------------------------------
struct BwdParams {
    int n;
    long long q0;
    int Hq, Hkv;
    const float *lse;     // [Hq, n]
    const float *delta;   // [Hq, n]
    float *dq;            // [n, Hq, 128]
    float *dk, *dv;       // [q0 + n, Hkv, 128]
    float scale, scale_log2;
};

constexpr int KV_QSTAGES = 3;
constexpr int BWD_ALIGN_SLACK = 768;    // what the 227 KB carve-out leaves for aligning the tiles to 1024 bytes
constexpr int BWD_SMEM = (4 + KV_QSTAGES) * TILE_BYTES + 4 * TILE * 4 /* lse, delta x 2 stages */ + 256 + BWD_ALIGN_SLACK;
static_assert(BWD_SMEM <= 232448, "dK/dV role exceeds the shared memory of an SM");
constexpr int DQ_KSTAGES = 3;
constexpr int DQ_SMEM = (4 + DQ_KSTAGES) * TILE_BYTES + 1024 + 256;   // Q, dO, K x 3, V x 2
constexpr int BWD_THREADS = 64 + 512;
constexpr int HALF = 64;

__device__ __forceinline__ void abort_drain(volatile int *abort_flag) {
    if (*abort_flag) {   // give copies that are still in flight time to land before shared memory is released
        const unsigned long long t0 = global_timer();
        while (global_timer() - t0 < 200000ull) { }
    }
}

__device__ __forceinline__ void attn_bwd_dkdv_body(const CUtensorMap &map_q, const CUtensorMap &map_k,
                                                   const CUtensorMap &map_v, const CUtensorMap &map_do,
                                                   const BwdParams &p, uint8_t *smem_raw, int block_x, int block_y) {
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const uint32_t sK = base, sV = sK + TILE_BYTES, sQ = sV + TILE_BYTES, sdO = sQ + KV_QSTAGES * TILE_BYTES;
    uint8_t *tail = smem_raw + (base - raw) + (4 + KV_QSTAGES) * TILE_BYTES;
    float *s_lse = reinterpret_cast<float *>(tail);           // [2][128], pre-multiplied by log2(e)
    float *s_delta = s_lse + 2 * TILE;                        // [2][128], pre-multiplied by the score scale
    uint8_t *aux = tail + 4 * TILE * 4;
    const uint32_t bars = smem_u32(aux);
    const uint32_t kv_full = bars, q_full = bars + 8, q_empty = bars + 32, do_full = bars + 56, do_empty = bars + 72,
                   rows_empty = bars + 88, s_full = bars + 104, dp_full = bars + 112, loaded = bars + 120,
                   p1_full = bars + 128, p2_full = bars + 136, acc_full = bars + 144;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(aux + 152);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(aux + 160);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = block_y, G = p.Hq / p.Hkv;
    const long long k_abs0 = (long long)block_x * TILE;
    const int nqt = (p.n + TILE - 1) / TILE;
    const int first_qt = k_abs0 > p.q0 ? (int)((k_abs0 - p.q0) / TILE) : 0;
    const int per_head = nqt - first_qt;
    const int iters = G * per_head;

    if (threadIdx.x == 0) {
        mbar_init(kv_full, 1);
        for (int s = 0; s < KV_QSTAGES; s++) {
            mbar_init(q_full + 8 * s, 1);
            mbar_init(q_empty + 8 * s, 1);
        }
        for (int s = 0; s < 2; s++) {
            mbar_init(do_full + 8 * s, 1);
            mbar_init(do_empty + 8 * s, 1);
            mbar_init(rows_empty + 8 * s, 1);
        }
        mbar_init(s_full, 1);
        mbar_init(dp_full, 1);
        mbar_init(loaded, 16);
        mbar_init(p1_full, 16);
        mbar_init(p2_full, 16);
        mbar_init(acc_full, 1);
        // the carve-out leaves at most 768 bytes for aligning the tiles to 1024: a base that needs more cannot be used
        *abort_flag = (base - raw) > BWD_ALIGN_SLACK ? 1 : 0;
        if (*abort_flag) atomicExch(&g_tc_fault, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    // columns: S^T at 0; dP^T at 128, later P^T (packed) in the first and dS^T (packed) in the second 16 columns of
    // every 32-column group; dV at 256, dK at 384
    const uint32_t tST = tmem, tDPT = tmem + 128, tDV = tmem + 256, tDK = tmem + 384;
    const bool usable = *abort_flag == 0;

    if (!usable) {
        // nothing was issued: fall through to the common exit
    } else if (warp == 0) {
        // ---- producer: K, V once; per iteration the dO tile with the lse / delta rows (two stages) and the Q tile
        // (three stages: Q_i is read by S^T_i, which is issued a whole iteration ahead, and again by dK_i at the end)
        if (lane == 0) {
            mbar_expect_tx(kv_full, 2 * TILE_BYTES);
            tma_load_2d(sK, &map_k, kv_full, g * TILE, (int)k_abs0);
            tma_load_2d(sK + HALF_BYTES, &map_k, kv_full, g * TILE + 64, (int)k_abs0);
            tma_load_2d(sV, &map_v, kv_full, g * TILE, (int)k_abs0);
            tma_load_2d(sV + HALF_BYTES, &map_v, kv_full, g * TILE + 64, (int)k_abs0);
        }
        uint32_t sq = 0, qph = 0;
        for (int it = 0; it < iters; it++) {
            const int h = g * G + it / per_head, qt0 = (first_qt + it % per_head) * TILE;
            const uint32_t sd = it & 1, dph = (it >> 1) & 1;
            int ok = 1;
            if (lane == 0) {
                ok = mbar_wait(q_empty + 8 * sq, qph ^ 1u, abort_flag) ? 1 : 0;          // dK of the stage's last user
                if (ok) {
                    mbar_expect_tx(q_full + 8 * sq, TILE_BYTES);
                    tma_load_2d(sQ + sq * TILE_BYTES, &map_q, q_full + 8 * sq, h * TILE, qt0);
                    tma_load_2d(sQ + sq * TILE_BYTES + HALF_BYTES, &map_q, q_full + 8 * sq, h * TILE + 64, qt0);
                    ok = mbar_wait(do_empty + 8 * sd, dph ^ 1u, abort_flag) ? 1 : 0;     // dV of the stage's last user
                }
                if (ok) {
                    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(do_full + 8 * sd), "r"(TILE_BYTES) : "memory");
                    tma_load_2d(sdO + sd * TILE_BYTES, &map_do, do_full + 8 * sd, h * TILE, qt0);
                    tma_load_2d(sdO + sd * TILE_BYTES + HALF_BYTES, &map_do, do_full + 8 * sd, h * TILE + 64, qt0);
                    ok = mbar_wait(rows_empty + 8 * sd, dph ^ 1u, abort_flag) ? 1 : 0;   // delta rows: read until dS^T is packed
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
#pragma unroll
            for (int e = 0; e < 4; e++) {
                const int col = lane * 4 + e, r = qt0 + col;
                s_lse[sd * TILE + col] = r < p.n ? p.lse[(long long)h * p.n + r] * kLog2e : 0.f;
                s_delta[sd * TILE + col] = r < p.n ? p.delta[(long long)h * p.n + r] * p.scale : 0.f;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(do_full + 8 * sd);   // publishes the rows; the phase completes when dO has landed too
            if (++sq == KV_QSTAGES) { sq = 0; qph ^= 1u; }
        }
    }
    else if (warp == 1) {
        // the whole warp runs the issue loop; each MMA / commit executes in one elected lane
        constexpr uint32_t idesc_kk = make_idesc(TILE, TILE, false, false);     // both operands K-major
        constexpr uint32_t idesc_acc = make_idesc(TILE, TILE, false, true);     // B MN-major (N = head dims)
        bool alive = mbar_wait_warp(kv_full, 0, abort_flag);
        const uint32_t k_lo = klo(sK), v_lo = klo(sV);
        uint32_t sq_s = 0, qph_s = 0;      // Q stage / phase of the next S^T
        uint32_t sq_k = 0;                 // Q stage of the next dK
        auto issue_st = [&]() -> bool {    // S^T = K Q^T for the next iteration
            if (!mbar_wait_warp(q_full + 8 * sq_s, qph_s, abort_flag)) return false;
            tc_fence_after();
            const uint32_t q_lo = klo(sQ + sq_s * TILE_BYTES);
#pragma unroll
            for (int kk = 0; kk < 8; kk++) umma_ss_w(tST, k_lo + kstep(kk), q_lo + kstep(kk), idesc_kk, kk != 0);
            umma_commit_w(s_full);
            if (++sq_s == KV_QSTAGES) { sq_s = 0; qph_s ^= 1u; }
            return true;
        };
        auto issue_dpt = [&](int it) -> bool {     // dP^T = V dO^T of iteration `it`
            if (!mbar_wait_warp(do_full + 8 * (it & 1), (it >> 1) & 1, abort_flag)) return false;
            tc_fence_after();
            const uint32_t do_lo = klo(sdO + (it & 1) * TILE_BYTES);
#pragma unroll
            for (int kk = 0; kk < 8; kk++) umma_ss_w(tDPT, v_lo + kstep(kk), do_lo + kstep(kk), idesc_kk, kk != 0);
            umma_commit_w(dp_full);
            return true;
        };
        if (alive && iters > 0) alive = issue_st() && issue_dpt(0);
        for (int it = 0; it < iters && alive; it++) {
            const uint32_t sd = it & 1;
            // the softmax warps hold S^T_it in registers: its columns take S^T of the next iteration at once
            if (it + 1 < iters) {
                if (!mbar_wait_warp(loaded, it & 1, abort_flag)) { alive = false; break; }
                tc_fence_after();
                if (!issue_st()) { alive = false; break; }
            }
            // dV += P^T dO as soon as P^T is packed (first 16 columns of each group of the dP^T region)
            if (!mbar_wait_warp(p1_full, it & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
            const uint32_t do_mn = mnlo(sdO + sd * TILE_BYTES);
#pragma unroll
            for (int kk = 0; kk < 8; kk++)
                umma_ts_w(tDV, tDPT + (kk >> 1) * 32 + (kk & 1) * 8, do_mn + mnstep(kk), idesc_acc, (it | kk) != 0);
            umma_commit_w(do_empty + 8 * sd);            // dO of this stage is consumed (dP^T was issued earlier)
            // dK += dS^T Q (second 16 columns of each group)
            if (!mbar_wait_warp(p2_full, it & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
            const uint32_t q_mn = mnlo(sQ + sq_k * TILE_BYTES);
#pragma unroll
            for (int kk = 0; kk < 8; kk++)
                umma_ts_w(tDK, tDPT + (kk >> 1) * 32 + 16 + (kk & 1) * 8, q_mn + mnstep(kk), idesc_acc, (it | kk) != 0);
            umma_commit_w(q_empty + 8 * sq_k);           // Q of this stage is consumed
            umma_commit_w(rows_empty + 8 * sd);          // and so are the lse / delta rows
            if (++sq_k == KV_QSTAGES) sq_k = 0;
            // the dP^T region is free once dV and dK have read it (in order): next iteration's dP^T
            if (it + 1 < iters && !issue_dpt(it + 1)) { alive = false; break; }
        }
        if (alive) umma_commit_w(acc_full);
    }
    else {
        const int quarter = warp & 3;
        const int wg = (warp - 2) >> 2;                           // 0..3: 32-query group of the tile
        const int col_base = wg * 32;
        const int row = quarter * 32 + lane;                      // key row within the tile
        const long long k_abs = k_abs0 + row;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        // The group reads its 32 fp32 columns of S^T and of dP^T into registers, then writes the packed bf16 pairs
        // of P^T over the first and of dS^T over the second 16 of ITS OWN dP^T columns; the MMA thread addresses
        // each 16-query slice of those A operands separately.  S^T's columns are never written by these warps, so
        // the product of the next iteration can refill them while this iteration's exponentials are computed.
        const uint32_t tS_g = tST + col_base + lane_base, tP_g = tDPT + col_base + lane_base;
        bool alive = true;
        for (int it = 0; it < iters && alive; it++) {
            const int qt0 = (first_qt + it % per_head) * TILE;
            const uint32_t sd = it & 1;
            if (!mbar_wait(s_full, it & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
            uint32_t rs[32];
            tmem_ld32(tS_g, rs);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(loaded);
            // the producer's lse / delta rows of this stage are published together with the dO tile
            if (!mbar_wait(do_full + 8 * sd, (it >> 1) & 1, abort_flag)) { alive = false; break; }
            const long long q_abs0 = p.q0 + qt0;
            const bool diag = k_abs0 + TILE - 1 > q_abs0;          // the tile pair holds masked (query, key) pairs
            // query column c of the tile is visible to this key iff q_abs0 + c >= k_abs
            const int first_col = (k_abs > q_abs0) ? (int)((k_abs - q_abs0) > TILE ? TILE : (k_abs - q_abs0)) : 0;
            const float *lse2 = s_lse + sd * TILE + col_base, *dl = s_delta + sd * TILE + col_base;
            // phase 1: P^T = exp2(S^T * scale - lse), all the dV product needs
            float pv[32];
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
                const float4 l4 = *reinterpret_cast<const float4 *>(lse2 + e);
                const float lv[4] = {l4.x, l4.y, l4.z, l4.w};
#pragma unroll
                for (int t = 0; t < 4; t++) {
                    float x = fmaf(__uint_as_float(rs[e + t]), p.scale_log2, -lv[t]);
                    if (diag && col_base + e + t < first_col) x = -INFINITY;
                    pv[e + t] = fast_exp2(x);
                }
            }
            // dP^T of this iteration was queued a whole iteration ago; its columns become P^T and dS^T
            uint32_t pp[16];
#pragma unroll
            for (int e = 0; e < 32; e += 2) pp[e / 2] = pack_bf16(pv[e], pv[e + 1]);
            if (!mbar_wait(dp_full, it & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
            uint32_t rp[32];
            tmem_ld32(tP_g, rp);
            {
                tmem_st16(tP_g, pp);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(p1_full);
            }
            // phase 2: dS^T = P^T * (dP^T * scale - delta * scale)
            {
                uint32_t ds[16];
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    const float4 d4 = *reinterpret_cast<const float4 *>(dl + e);
                    const float dv[4] = {d4.x, d4.y, d4.z, d4.w};
                    float dsv[4];
#pragma unroll
                    for (int t = 0; t < 4; t++) dsv[t] = pv[e + t] * fmaf(__uint_as_float(rp[e + t]), p.scale, -dv[t]);
                    ds[e / 2] = pack_bf16(dsv[0], dsv[1]);
                    ds[e / 2 + 1] = pack_bf16(dsv[2], dsv[3]);
                }
                tmem_st16(tP_g + 16, ds);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(p2_full);
            }
        }
        if (alive && mbar_wait(acc_full, 0, abort_flag)) {
            tc_fence_after();
            const bool in_range = k_abs < p.q0 + p.n;
            // group wg writes head dims 32*wg .. 32*wg+31
            uint32_t rv[32], rk[32];
            tmem_ld32(tDV + lane_base + col_base, rv);
            tmem_ld32(tDK + lane_base + col_base, rk);
            if (in_range) {
                float *pv = p.dv + (k_abs * p.Hkv + g) * TILE + col_base;
                float *pk = p.dk + (k_abs * p.Hkv + g) * TILE + col_base;
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    float4 a = *reinterpret_cast<float4 *>(pv + e);
                    a.x += __uint_as_float(rv[e]); a.y += __uint_as_float(rv[e + 1]);
                    a.z += __uint_as_float(rv[e + 2]); a.w += __uint_as_float(rv[e + 3]);
                    *reinterpret_cast<float4 *>(pv + e) = a;
                    float4 b = *reinterpret_cast<float4 *>(pk + e);
                    b.x += __uint_as_float(rk[e]); b.y += __uint_as_float(rk[e + 1]);
                    b.z += __uint_as_float(rk[e + 2]); b.w += __uint_as_float(rk[e + 3]);
                    *reinterpret_cast<float4 *>(pk + e) = b;
                }
            }
        }
    }

    __syncwarp();
    abort_drain(abort_flag);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, 512);
    }
}

__device__ __forceinline__ void attn_bwd_dq_body(const CUtensorMap &map_q, const CUtensorMap &map_k,
                                                 const CUtensorMap &map_v, const CUtensorMap &map_do,
                                                 const BwdParams &p, uint8_t *smem_raw, int block_x, int block_y) {
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    // K tiles live from S_j to dQ_j, so their ring has three stages: the copy of tile j+2 then starts when dQ of
    // tile j-1 is done and its latency hides behind a whole tile of work.  V tiles are released right after dP_j.
    const uint32_t sQ = base, sdO = sQ + TILE_BYTES, sK = sdO + TILE_BYTES, sV = sK + DQ_KSTAGES * TILE_BYTES;
    uint8_t *aux = smem_raw + (base - raw) + (4 + DQ_KSTAGES) * TILE_BYTES;
    const uint32_t bars = smem_u32(aux);
    const uint32_t q_full = bars, k_full = bars + 8, k_empty = bars + 32, v_full = bars + 56, v_empty = bars + 72,
                   s_full = bars + 88, dp_full = bars + 96, s_free = bars + 104, p2_full = bars + 112,
                   acc_full = bars + 120;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(aux + 128);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(aux + 136);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = block_y, g = h / (p.Hq / p.Hkv);
    const int qt0 = block_x * TILE;
    const long long q_abs0 = p.q0 + qt0;
    const int rows_here = (p.n - qt0) < TILE ? (p.n - qt0) : TILE;
    const long long kv_end = q_abs0 + rows_here;
    const int nkv = (int)((kv_end + TILE - 1) / TILE);

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < DQ_KSTAGES; s++) {
            mbar_init(k_full + 8 * s, 1);
            mbar_init(k_empty + 8 * s, 1);
        }
        for (int s = 0; s < 2; s++) {
            mbar_init(v_full + 8 * s, 1);
            mbar_init(v_empty + 8 * s, 1);
        }
        mbar_init(s_full, 1);
        mbar_init(dp_full, 1);
        mbar_init(s_free, 16);
        mbar_init(p2_full, 16);
        mbar_init(acc_full, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    // columns: S at 0, dP at 128, dQ at 256
    const uint32_t tS = tmem, tDP = tmem + 128, tDQ = tmem + 256;

    if (warp == 0) {
        if (lane == 0) {
            mbar_expect_tx(q_full, 2 * TILE_BYTES);
            tma_load_2d(sQ, &map_q, q_full, h * TILE, qt0);
            tma_load_2d(sQ + HALF_BYTES, &map_q, q_full, h * TILE + 64, qt0);
            tma_load_2d(sdO, &map_do, q_full, h * TILE, qt0);
            tma_load_2d(sdO + HALF_BYTES, &map_do, q_full, h * TILE + 64, qt0);
            uint32_t ks = 0, kph = 0;
            for (int j = 0; j < nkv; j++) {
                if (!mbar_wait(k_empty + 8 * ks, kph ^ 1u, abort_flag)) break;
                mbar_expect_tx(k_full + 8 * ks, TILE_BYTES);
                tma_load_2d(sK + ks * TILE_BYTES, &map_k, k_full + 8 * ks, g * TILE, j * TILE);
                tma_load_2d(sK + ks * TILE_BYTES + HALF_BYTES, &map_k, k_full + 8 * ks, g * TILE + 64, j * TILE);
                if (++ks == DQ_KSTAGES) { ks = 0; kph ^= 1u; }
                const uint32_t vs = j & 1, vph = (j >> 1) & 1;
                if (!mbar_wait(v_empty + 8 * vs, vph ^ 1u, abort_flag)) break;
                mbar_expect_tx(v_full + 8 * vs, TILE_BYTES);
                tma_load_2d(sV + vs * TILE_BYTES, &map_v, v_full + 8 * vs, g * TILE, j * TILE);
                tma_load_2d(sV + vs * TILE_BYTES + HALF_BYTES, &map_v, v_full + 8 * vs, g * TILE + 64, j * TILE);
            }
        }
    } else if (warp == 1) {
        // the whole warp runs the issue loop; each MMA / commit executes in one elected lane
        constexpr uint32_t idesc_kk = make_idesc(TILE, TILE, false, false);
        constexpr uint32_t idesc_acc = make_idesc(TILE, TILE, false, true);
        bool alive = mbar_wait_warp(q_full, 0, abort_flag);
        const uint32_t q_lo = klo(sQ), do_lo = klo(sdO);
        // K stage and phase of the tile whose S is issued next / whose dQ is issued next
        uint32_t ks_s = 0, kph_s = 0, ks_q = 0;
        auto issue_s = [&](int j) -> bool {        // S = Q K^T
            (void)j;
            if (!mbar_wait_warp(k_full + 8 * ks_s, kph_s, abort_flag)) return false;
            tc_fence_after();
            const uint32_t k_lo = klo(sK + ks_s * TILE_BYTES);
#pragma unroll
            for (int kk = 0; kk < 8; kk++) umma_ss_w(tS, q_lo + kstep(kk), k_lo + kstep(kk), idesc_kk, kk != 0);
            umma_commit_w(s_full);
            if (++ks_s == DQ_KSTAGES) { ks_s = 0; kph_s ^= 1u; }
            return true;
        };
        auto issue_dp = [&](int j) -> bool {       // dP = dO V^T
            const uint32_t vs = j & 1;
            if (!mbar_wait_warp(v_full + 8 * vs, (j >> 1) & 1, abort_flag)) return false;
            tc_fence_after();
            const uint32_t v_lo = klo(sV + vs * TILE_BYTES);
#pragma unroll
            for (int kk = 0; kk < 8; kk++) umma_ss_w(tDP, do_lo + kstep(kk), v_lo + kstep(kk), idesc_kk, kk != 0);
            umma_commit_w(v_empty + 8 * vs);             // V of this stage is consumed
            umma_commit_w(dp_full);
            return true;
        };
        if (alive) alive = issue_s(0) && issue_dp(0);
        for (int j = 0; j < nkv && alive; j++) {
            if (j + 1 < nkv) {
                // next tile's S as soon as the softmax warps have read this tile's S into registers
                if (!mbar_wait_warp(s_free, j & 1, abort_flag)) { alive = false; break; }
                tc_fence_after();
                if (!issue_s(j + 1)) { alive = false; break; }
            }
            if (!mbar_wait_warp(p2_full, j & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
            const uint32_t k_mn = mnlo(sK + ks_q * TILE_BYTES);
#pragma unroll
            for (int kk = 0; kk < 8; kk++)
                umma_ts_w(tDQ, tDP + (kk >> 1) * 32 + (kk & 1) * 8, k_mn + mnstep(kk), idesc_acc, (j | kk) != 0);
            umma_commit_w(k_empty + 8 * ks_q);           // K of this stage is consumed
            if (++ks_q == DQ_KSTAGES) ks_q = 0;
            // the dP columns are free once dQ has read dS (in order)
            if (j + 1 < nkv && !issue_dp(j + 1)) { alive = false; break; }
        }
        if (alive) umma_commit_w(acc_full);
    } else {
        const int quarter = warp & 3;
        const int wg = (warp - 2) >> 2;                           // 0..3: 32-key group of the tile
        const int key_base = wg * 32;
        const int row = quarter * 32 + lane;
        const int qr = qt0 + row;
        const long long q_abs = q_abs0 + row;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        const uint32_t tS_g = tS + key_base + lane_base, tP_g = tDP + key_base + lane_base;
        const float neg_lse2 = qr < p.n ? -p.lse[(long long)h * p.n + qr] * kLog2e : 0.f;
        const float neg_delta_s = qr < p.n ? -p.delta[(long long)h * p.n + qr] * p.scale : 0.f;
        bool alive = true;
        for (int j = 0; j < nkv && alive; j++) {
            if (!mbar_wait(s_full, j & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
            const long long k_abs0 = (long long)j * TILE;
            const bool diag = k_abs0 + TILE - 1 > q_abs0;
            const int lim = (int)(q_abs - k_abs0);                // keys 0..lim of the tile are visible (diag tiles)
            // phase 1: P from S; the S columns are handed back to the tensor pipe right after the load
            float pv[32];
            {
                uint32_t rs[32];
                tmem_ld32(tS_g, rs);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(s_free);
#pragma unroll
                for (int e = 0; e < 32; e++) {
                    float x = fmaf(__uint_as_float(rs[e]), p.scale_log2, neg_lse2);
                    if (diag && key_base + e > lim) x = -INFINITY;
                    pv[e] = fast_exp2(x);
                }
            }
            // phase 2: dS = P * (dP * scale - delta * scale), packed in place
            if (!mbar_wait(dp_full, j & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
            {
                uint32_t rp[32], ds[16];
                tmem_ld32(tP_g, rp);
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    const float d0 = pv[e] * fmaf(__uint_as_float(rp[e]), p.scale, neg_delta_s);
                    const float d1 = pv[e + 1] * fmaf(__uint_as_float(rp[e + 1]), p.scale, neg_delta_s);
                    ds[e / 2] = pack_bf16(d0, d1);
                }
                tmem_st16(tP_g, ds);       // front of the group's own fp32 columns
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(p2_full);
            }
        }
        if (alive && mbar_wait(acc_full, 0, abort_flag)) {
            tc_fence_after();
            uint32_t r[32];
            tmem_ld32(tDQ + lane_base + key_base, r);
            if (qr < p.n) {
                float *out = p.dq + ((long long)qr * p.Hq + h) * TILE + key_base;
#pragma unroll
                for (int e = 0; e < 32; e += 4)
                    *reinterpret_cast<float4 *>(out + e) =
                        make_float4(__uint_as_float(r[e]), __uint_as_float(r[e + 1]), __uint_as_float(r[e + 2]),
                                    __uint_as_float(r[e + 3]));
            }
        }
    }

    __syncwarp();
    abort_drain(abort_flag);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, 512);
    }
}


// ---------------------------------------------------------------------------------------------
// Five-product backward: the key-tile owners also form dQ.  One role only (the dK/dV role above plus one
// product): per tile pair dQ^T_partial = K^T dS^T lands in the dP^T region once dV and dK have read P^T and dS^T
// from it, four drain warps add it into the fp32 dQ in global memory (L2-resident: [chunk, Hq, 128] floats), and
// the region then takes dP^T of the next iteration.  dS^T reaches that product through shared memory (the softmax
// warps write their row segments in the swizzled tile layout), next to its packed copy in tensor memory for dK.
// Five executed products per tile pair instead of seven.  The adds of different key tiles into one dQ tile arrive in
// whatever order the CTAs run, so dQ is NOT bit-reproducible from run to run (dK and dV are): an opt-in variant,
// not what the layer uses.  Measured (2048 queries, 16384-key prefix, back to back for seconds at the power limit):
// 1.73 ms per call against 1.81 ms for the two-role kernel; 1.54 vs 1.57 ms in a burst.  An iteration takes ~5900
// cycles here against ~3200 + ~2550 for the two roles; what bounds it is shared-memory traffic (~540 KB per
// iteration: five products' operands, the incoming Q / dO tiles, dS^T and the drain's staging) and the rate at which
// L2 takes the reduce-adds (64 KB per tile pair) while it also serves the K / V / Q / dO stream.
// ---------------------------------------------------------------------------------------------
constexpr int FUSED_QSTAGES = 2;
constexpr int FUSED_DRAIN_WARP0 = 18;
constexpr int FUSED_THREADS = (FUSED_DRAIN_WARP0 + 4) * 32;
static_assert((5 + FUSED_QSTAGES) * TILE_BYTES + 4 * TILE * 4 + 256 + BWD_ALIGN_SLACK <= 232448, "fused role exceeds shared memory");

__device__ __forceinline__ void attn_bwd_fused_body(const CUtensorMap &map_q, const CUtensorMap &map_k,
                                                   const CUtensorMap &map_v, const CUtensorMap &map_do,
                                                   const CUtensorMap &map_dq, const BwdParams &p, uint8_t *smem_raw, int block_x, int block_y) {
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    // K, V (resident), Q x 2, dO x 1 (its successor is fetched while dK, dQ and the drain run), dS^T, and 32 KiB of
    // staging for the drain warps
    const uint32_t sK = base, sV = sK + TILE_BYTES, sQ = sV + TILE_BYTES, sdO = sQ + FUSED_QSTAGES * TILE_BYTES,
                   sdS = sdO + TILE_BYTES, sStage = sdS + TILE_BYTES;
    uint8_t *tail = smem_raw + (base - raw) + (5 + FUSED_QSTAGES) * TILE_BYTES;
    float *s_lse = reinterpret_cast<float *>(tail);           // [2][128], pre-multiplied by log2(e)
    float *s_delta = s_lse + 2 * TILE;                        // [2][128], pre-multiplied by the score scale
    uint8_t *aux = tail + 4 * TILE * 4;
    const uint32_t bars = smem_u32(aux);
    const uint32_t kv_full = bars, q_full = bars + 8, q_empty = bars + 32, do_full = bars + 56, do_empty = bars + 64,
                   rows_full = bars + 72, rows_empty = bars + 88, s_full = bars + 104, dp_full = bars + 112, loaded = bars + 120,
                   p1_full = bars + 128, p2_full = bars + 136, acc_full = bars + 144, dq_full = bars + 152,
                   b_free = bars + 160, p3_full = bars + 176;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(aux + 184);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(aux + 192);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = block_y, G = p.Hq / p.Hkv;
    const long long k_abs0 = (long long)block_x * TILE;
    const int nqt = (p.n + TILE - 1) / TILE;
    const int first_qt = k_abs0 > p.q0 ? (int)((k_abs0 - p.q0) / TILE) : 0;
    const int per_head = nqt - first_qt;
    const int iters = G * per_head;
    // CTAs that run at the same time (neighbouring key tiles) start their walk over the (head, query tile) pairs at
    // different places, so that their adds into dQ do not all go to the same tile at once (no measurable effect on
    // the time; kept because it costs nothing)
    const int rot = (int)(((long long)block_x * 37) % iters);

    if (threadIdx.x == 0) {
        mbar_init(kv_full, 1);
        for (int s = 0; s < FUSED_QSTAGES; s++) {
            mbar_init(q_full + 8 * s, 1);
            mbar_init(q_empty + 8 * s, 1);
        }
        mbar_init(do_full, 1);
        mbar_init(do_empty, 1);
        for (int s = 0; s < 2; s++) {
            mbar_init(rows_full + 8 * s, 1);
            mbar_init(rows_empty + 8 * s, 1);
        }
        mbar_init(s_full, 1);
        mbar_init(dp_full, 1);
        mbar_init(loaded, 16);
        mbar_init(p1_full, 16);
        mbar_init(p2_full, 16);
        mbar_init(acc_full, 1);
        mbar_init(dq_full, 1);
        mbar_init(b_free, 4);
        mbar_init(p3_full, 16);
        // the carve-out leaves at most 768 bytes for aligning the tiles to 1024: a base that needs more cannot be used
        *abort_flag = (base - raw) > BWD_ALIGN_SLACK ? 1 : 0;
        if (*abort_flag) atomicExch(&g_tc_fault, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    // columns: S^T at 0; dP^T at 128, later P^T (packed) in the first and dS^T (packed) in the second 16 columns of
    // every 32-column group, and then this tile pair's share of dQ (queries on the lanes); dV at 256, dK at 384
    const uint32_t tST = tmem, tDPT = tmem + 128, tDV = tmem + 256, tDK = tmem + 384;
    const bool usable = *abort_flag == 0;

    if (!usable) {
        // nothing was issued: fall through to the common exit
    } else if (warp == 0) {
        // ---- producer: K, V once; per iteration the Q tile (two stages), the dO tile (one: its successor is fetched
        // as soon as dV has read it) and the lse / delta rows (two stages)
        if (lane == 0) {
            mbar_expect_tx(kv_full, 2 * TILE_BYTES);
            tma_load_2d(sK, &map_k, kv_full, g * TILE, (int)k_abs0);
            tma_load_2d(sK + HALF_BYTES, &map_k, kv_full, g * TILE + 64, (int)k_abs0);
            tma_load_2d(sV, &map_v, kv_full, g * TILE, (int)k_abs0);
            tma_load_2d(sV + HALF_BYTES, &map_v, kv_full, g * TILE + 64, (int)k_abs0);
        }
        uint32_t sq = 0, qph = 0;
        for (int it = 0; it < iters; it++) {
            const int il = (it + rot) % iters, h = g * G + il / per_head, qt0 = (first_qt + il % per_head) * TILE;
            const uint32_t sd = it & 1, dph = (it >> 1) & 1;
            int ok = 1;
            if (lane == 0) {
                ok = mbar_wait(q_empty + 8 * sq, qph ^ 1u, abort_flag) ? 1 : 0;          // dK of the stage's last user
                if (ok) {
                    mbar_expect_tx(q_full + 8 * sq, TILE_BYTES);
                    tma_load_2d(sQ + sq * TILE_BYTES, &map_q, q_full + 8 * sq, h * TILE, qt0);
                    tma_load_2d(sQ + sq * TILE_BYTES + HALF_BYTES, &map_q, q_full + 8 * sq, h * TILE + 64, qt0);
                    ok = mbar_wait(do_empty, (uint32_t)(it & 1) ^ 1u, abort_flag) ? 1 : 0;   // dV of the previous iteration
                }
                if (ok) {
                    mbar_expect_tx(do_full, TILE_BYTES);
                    tma_load_2d(sdO, &map_do, do_full, h * TILE, qt0);
                    tma_load_2d(sdO + HALF_BYTES, &map_do, do_full, h * TILE + 64, qt0);
                    ok = mbar_wait(rows_empty + 8 * sd, dph ^ 1u, abort_flag) ? 1 : 0;   // delta rows: read until dS^T is packed
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
#pragma unroll
            for (int e = 0; e < 4; e++) {
                const int col = lane * 4 + e, r = qt0 + col;
                s_lse[sd * TILE + col] = r < p.n ? p.lse[(long long)h * p.n + r] * kLog2e : 0.f;
                s_delta[sd * TILE + col] = r < p.n ? p.delta[(long long)h * p.n + r] * p.scale : 0.f;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(rows_full + 8 * sd);   // publishes the rows
            if (++sq == FUSED_QSTAGES) { sq = 0; qph ^= 1u; }
        }
    }
    else if (warp == 1) {
        // the whole warp runs the issue loop; each MMA / commit executes in one elected lane
        constexpr uint32_t idesc_kk = make_idesc(TILE, TILE, false, false);     // both operands K-major
        constexpr uint32_t idesc_acc = make_idesc(TILE, TILE, false, true);     // B MN-major (N = head dims)
        constexpr uint32_t idesc_tt = make_idesc(TILE, TILE, true, true);       // both MN-major (contraction along rows)
        bool alive = mbar_wait_warp(kv_full, 0, abort_flag);
        const uint32_t k_lo = klo(sK), v_lo = klo(sV), k_mn = mnlo(sK), ds_mn = mnlo(sdS);
        uint32_t sq_s = 0, qph_s = 0;      // Q stage / phase of the next S^T
        uint32_t sq_k = 0;                 // Q stage of the next dK
        auto issue_st = [&]() -> bool {    // S^T = K Q^T for the next iteration
            if (!mbar_wait_warp(q_full + 8 * sq_s, qph_s, abort_flag)) return false;
            tc_fence_after();
            const uint32_t q_lo = klo(sQ + sq_s * TILE_BYTES);
#pragma unroll
            for (int kk = 0; kk < 8; kk++) umma_ss_w(tST, k_lo + kstep(kk), q_lo + kstep(kk), idesc_kk, kk != 0);
            umma_commit_w(s_full);
            if (++sq_s == FUSED_QSTAGES) { sq_s = 0; qph_s ^= 1u; }
            return true;
        };
        auto issue_dpt = [&](int it) -> bool {     // dP^T = V dO^T of iteration `it`
            if (!mbar_wait_warp(do_full, it & 1, abort_flag)) return false;
            tc_fence_after();
            const uint32_t do_lo = klo(sdO);
#pragma unroll
            for (int kk = 0; kk < 8; kk++) umma_ss_w(tDPT, v_lo + kstep(kk), do_lo + kstep(kk), idesc_kk, kk != 0);
            umma_commit_w(dp_full);
            return true;
        };
        if (alive && iters > 0) alive = issue_st() && issue_dpt(0);
        for (int it = 0; it < iters && alive; it++) {
            const uint32_t sd = it & 1;
            // the softmax warps hold S^T_it in registers: its columns take S^T of the next iteration at once
            if (it + 1 < iters) {
                if (!mbar_wait_warp(loaded, it & 1, abort_flag)) { alive = false; break; }
                tc_fence_after();
                if (!issue_st()) { alive = false; break; }
            }
            // dV += P^T dO as soon as P^T is packed (first 16 columns of each group of the dP^T region)
            if (!mbar_wait_warp(p1_full, it & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
            const uint32_t do_mn = mnlo(sdO);
#pragma unroll
            for (int kk = 0; kk < 8; kk++)
                umma_ts_w(tDV, tDPT + (kk >> 1) * 32 + (kk & 1) * 8, do_mn + mnstep(kk), idesc_acc, (it | kk) != 0);
            umma_commit_w(do_empty);                     // dO is consumed (dP^T was issued earlier): fetch the next one
            // dK += dS^T Q (second 16 columns of each group)
            if (!mbar_wait_warp(p2_full, it & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
            const uint32_t q_mn = mnlo(sQ + sq_k * TILE_BYTES);
#pragma unroll
            for (int kk = 0; kk < 8; kk++)
                umma_ts_w(tDK, tDPT + (kk >> 1) * 32 + 16 + (kk & 1) * 8, q_mn + mnstep(kk), idesc_acc, (it | kk) != 0);
            umma_commit_w(q_empty + 8 * sq_k);           // Q of this stage is consumed
            umma_commit_w(rows_empty + 8 * sd);          // and so are the lse / delta rows
            if (++sq_k == FUSED_QSTAGES) sq_k = 0;
            // this tile pair's share of dQ = dS K: both operands from shared memory with the contraction (the keys) along
            // their rows; it overwrites the dP^T region, which dV and dK (queued before it) have read by then
            if (!mbar_wait_warp(p3_full, it & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < 8; kk++)
                umma_ss_w(tDPT, ds_mn + mnstep(kk), k_mn + mnstep(kk), idesc_tt, kk != 0);
            umma_commit_w(dq_full);
            // the drain warps have the dQ share in registers: the region takes dP^T of the next iteration
            if (it + 1 < iters) {
                if (!mbar_wait_warp(b_free, it & 1, abort_flag)) { alive = false; break; }
                tc_fence_after();
                if (!issue_dpt(it + 1)) { alive = false; break; }
            }
        }
        if (alive) umma_commit_w(acc_full);
    }
    else if (warp >= FUSED_DRAIN_WARP0) {
        // ---- drain warps: this tile pair's share of dQ from tensor memory into the fp32 dQ in global memory, added
        // there by the copy engine (TMA reduce-add of 32 x 32 blocks staged in shared memory with the swizzle the
        // tensor map expects).  A warp owns 32 query rows (its lane quarter) and walks the four 32-column blocks; the
        // staging area is its own 8 KiB per warp: two rounds of two blocks, the second round's loads leave tensor memory
        // free while the first round's blocks are still being read by the copy engine.
        const int quarter = warp & 3;
        const uint32_t tD = tDPT + ((uint32_t)(quarter * 32) << 16);
        const uint32_t stage0 = sStage + (uint32_t)quarter * 8192u;     // two 4 KiB blocks per warp
        bool alive = true;
        for (int it = 0; it < iters && alive; it++) {
            const int il = (it + rot) % iters, h = g * G + il / per_head, qt0 = (first_qt + il % per_head) * TILE;
            if (!mbar_wait(dq_full, it & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
#pragma unroll 1
            for (int half = 0; half < 2; half++) {
                // 64 columns at a time: after the second load the whole block row is out of tensor memory
                uint32_t r[64];
                tmem_ld32_async(tD + half * 64, r);
                tmem_ld32_async(tD + half * 64 + 32, r + 32);
                tmem_wait_ld();
                if (half == 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(b_free);
                }
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // both staging blocks are free
                __syncwarp();
#pragma unroll
                for (int c = 0; c < 2; c++) {
                    const uint32_t buf_s = stage0 + c * 4096u;
#pragma unroll
                    for (int j = 0; j < 8; j++) {
                        const uint32_t dst = buf_s + lane * 128 + ((j ^ (lane & 7)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(r[32 * c + 4 * j]),
                                     "r"(r[32 * c + 4 * j + 1]), "r"(r[32 * c + 4 * j + 2]), "r"(r[32 * c + 4 * j + 3]) : "memory");
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) {
                    tma_reduce_add_2d(&map_dq, stage0, h * TILE + half * 64, qt0 + quarter * 32);   // rows past the chunk are clipped
                    tma_reduce_add_2d(&map_dq, stage0 + 4096u, h * TILE + half * 64 + 32, qt0 + quarter * 32);
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            }
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        __syncwarp();
    } else {
        const int quarter = warp & 3;
        const int wg = (warp - 2) >> 2;                           // 0..3: 32-query group of the tile
        const int col_base = wg * 32;
        const int row = quarter * 32 + lane;                      // key row within the tile
        const long long k_abs = k_abs0 + row;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        // The group reads its 32 fp32 columns of S^T and of dP^T into registers, then writes the packed bf16 pairs
        // of P^T over the first and of dS^T over the second 16 of ITS OWN dP^T columns; the MMA thread addresses
        // each 16-query slice of those A operands separately.  S^T's columns are never written by these warps, so
        // the product of the next iteration can refill them while this iteration's exponentials are computed.
        const uint32_t tS_g = tST + col_base + lane_base, tP_g = tDPT + col_base + lane_base;
        bool alive = true;
        for (int it = 0; it < iters && alive; it++) {
            const int qt0 = (first_qt + (it + rot) % iters % per_head) * TILE;
            const uint32_t sd = it & 1;
            if (!mbar_wait(s_full, it & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
            uint32_t rs[32];
            tmem_ld32(tS_g, rs);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(loaded);
            // the producer's lse / delta rows of this stage are published together with the dO tile
            if (!mbar_wait(rows_full + 8 * sd, (it >> 1) & 1, abort_flag)) { alive = false; break; }
            const long long q_abs0 = p.q0 + qt0;
            const bool diag = k_abs0 + TILE - 1 > q_abs0;          // the tile pair holds masked (query, key) pairs
            // query column c of the tile is visible to this key iff q_abs0 + c >= k_abs
            const int first_col = (k_abs > q_abs0) ? (int)((k_abs - q_abs0) > TILE ? TILE : (k_abs - q_abs0)) : 0;
            const float *lse2 = s_lse + sd * TILE + col_base, *dl = s_delta + sd * TILE + col_base;
            // phase 1: P^T = exp2(S^T * scale - lse), all the dV product needs
            float pv[32];
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
                const float4 l4 = *reinterpret_cast<const float4 *>(lse2 + e);
                const float lv[4] = {l4.x, l4.y, l4.z, l4.w};
#pragma unroll
                for (int t = 0; t < 4; t++) {
                    float x = fmaf(__uint_as_float(rs[e + t]), p.scale_log2, -lv[t]);
                    if (diag && col_base + e + t < first_col) x = -INFINITY;
                    pv[e + t] = fast_exp2(x);
                }
            }
            // dP^T of this iteration was queued a whole iteration ago; its columns become P^T and dS^T
            uint32_t pp[16];
#pragma unroll
            for (int e = 0; e < 32; e += 2) pp[e / 2] = pack_bf16(pv[e], pv[e + 1]);
            if (!mbar_wait(dp_full, it & 1, abort_flag)) { alive = false; break; }
            tc_fence_after();
            uint32_t rp[32];
            tmem_ld32(tP_g, rp);
            {
                tmem_st16(tP_g, pp);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(p1_full);
            }
            // phase 2: dS^T = P^T * (dP^T * scale - delta * scale)
            {
                uint32_t ds[16];
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    const float4 d4 = *reinterpret_cast<const float4 *>(dl + e);
                    const float dv[4] = {d4.x, d4.y, d4.z, d4.w};
                    float dsv[4];
#pragma unroll
                    for (int t = 0; t < 4; t++) dsv[t] = pv[e + t] * fmaf(__uint_as_float(rp[e + t]), p.scale, -dv[t]);
                    ds[e / 2] = pack_bf16(dsv[0], dsv[1]);
                    ds[e / 2 + 1] = pack_bf16(dsv[2], dsv[3]);
                }
                tmem_st16(tP_g + 16, ds);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(p2_full);          // dK may start; the dQ product waits for the copy below
                // the same dS^T row segment into shared memory for dQ = dS K: [128 keys][128 queries] bf16 as two
                // 64-query sub-tiles of 128-byte rows, 16-byte chunks swizzled by the row (what a TMA tile load leaves);
                // the buffer is free once the previous iteration's dQ product has read it
                if (it > 0 && !mbar_wait(dq_full, (it - 1) & 1, abort_flag)) { alive = false; break; }
                {
                    const uint32_t row_base = sdS + (uint32_t)(wg >> 1) * HALF_BYTES + (uint32_t)row * 128u;
#pragma unroll
                    for (int j = 0; j < 4; j++) {
                        const uint32_t chunk = (uint32_t)((wg & 1) * 4 + j) ^ (uint32_t)(row & 7);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row_base + (chunk << 4)), "r"(ds[4 * j]),
                                     "r"(ds[4 * j + 1]), "r"(ds[4 * j + 2]), "r"(ds[4 * j + 3]) : "memory");
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(p3_full);
            }
        }
        if (alive && mbar_wait(acc_full, 0, abort_flag)) {
            tc_fence_after();
            const bool in_range = k_abs < p.q0 + p.n;
            // group wg writes head dims 32*wg .. 32*wg+31
            uint32_t rv[32], rk[32];
            tmem_ld32(tDV + lane_base + col_base, rv);
            tmem_ld32(tDK + lane_base + col_base, rk);
            if (in_range) {
                float *pv = p.dv + (k_abs * p.Hkv + g) * TILE + col_base;
                float *pk = p.dk + (k_abs * p.Hkv + g) * TILE + col_base;
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    float4 a = *reinterpret_cast<float4 *>(pv + e);
                    a.x += __uint_as_float(rv[e]); a.y += __uint_as_float(rv[e + 1]);
                    a.z += __uint_as_float(rv[e + 2]); a.w += __uint_as_float(rv[e + 3]);
                    *reinterpret_cast<float4 *>(pv + e) = a;
                    float4 b = *reinterpret_cast<float4 *>(pk + e);
                    b.x += __uint_as_float(rk[e]); b.y += __uint_as_float(rk[e + 1]);
                    b.z += __uint_as_float(rk[e + 2]); b.w += __uint_as_float(rk[e + 3]);
                    *reinterpret_cast<float4 *>(pk + e) = b;
                }
            }
        }
    }

    __syncwarp();
    abort_drain(abort_flag);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, 512);
    }
}


__global__ void __launch_bounds__(FUSED_THREADS, 1)
    attn_bwd_fused_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                          const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do,
                          const __grid_constant__ CUtensorMap map_dq, const BwdParams p, int kv_tiles) {
    pdl_enter();
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const int b = (int)blockIdx.x;
    attn_bwd_fused_body(map_q, map_k, map_v, map_do, map_dq, p, smem_raw, b % kv_tiles, b / kv_tiles);
}

// One launch for both backward kernels.  They are independent (both read Q, K, V, dO, lse, delta; one owns dK / dV
// tiles, the other dQ tiles), and at short prefixes or small chunks neither fills the GPU on its own (e.g. 32 to
// 256 key-tile CTAs and 224 query-tile CTAs per chunk of the 7B layer at chunk 1024): as one grid their CTAs pack
// onto the SMs together.  The role whose CTAs run longest comes first (longest jobs first keeps the tail of the launch
// short): a dK / dV CTA walks G x (query tiles) tile pairs, a dQ CTA as many as its prefix has key tiles -- so the dQ
// CTAs lead at long prefixes and the dK / dV CTAs at short ones; within a role the longest CTAs come first too
// (lowest key tiles, highest query tiles).
constexpr int BWD_FUSED_SMEM = BWD_SMEM > DQ_SMEM ? BWD_SMEM : DQ_SMEM;
__global__ void __launch_bounds__(BWD_THREADS, 1)
    attn_bwd_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                       const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do,
                       const BwdParams p, int kv_tiles, int n_dkdv, int q_tiles, int n_dq_first) {
    pdl_enter();
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // block order = dispatch order: n_dq_first dQ CTAs (all of them or none), then the dK/dV CTAs, then the rest
    int b = (int)blockIdx.x;
    const bool dq_role = b < n_dq_first || b >= n_dq_first + n_dkdv;
    if (!dq_role) {
        b -= n_dq_first;
        // key tiles in ascending order, the KV heads of a key tile side by side: the cost of a CTA (the number of
        // query tiles that see its key tile) never increases along the list
        const int n_kv_heads = n_dkdv / kv_tiles;
        attn_bwd_dkdv_body(map_q, map_k, map_v, map_do, p, smem_raw, b / n_kv_heads, b % n_kv_heads);
    } else {
        const int c = b < n_dq_first ? b : b - n_dkdv;
        attn_bwd_dq_body(map_q, map_k, map_v, map_do, p, smem_raw, q_tiles - 1 - c % q_tiles, c / q_tiles);
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
                     float *lse, cudaStream_t st, int tiles_per_cta) {
    CUtensorMap mq, mk, mv;
    const int64_t kv_len = q0 + n;
    if (!make_tensor_map(&mq, q, n, (int64_t)Hq * TILE, (int64_t)Hq * TILE, 64, TILE, false) ||
        !make_tensor_map(&mk, k, kv_len, (int64_t)Hkv * TILE, (int64_t)Hkv * TILE, 64, TILE, false) ||
        !make_tensor_map(&mv, v, kv_len, (int64_t)Hkv * TILE, (int64_t)Hkv * TILE, 64, TILE, false))
        return STREAMBP_E_CUDA;
    static PerDevice configured;
    if (!configured.get([] { return opt_in_smem(attn_fwd_tc16_kernel, FWD16_SMEM) && opt_in_smem(attn_fwd_2q_kernel, FWD2Q_SMEM) ? 1 : 0; }))
        return STREAMBP_E_CUDA;
    FwdParams p{(int)n, (long long)q0, Hq, Hkv, o, lse, kLog2e / sqrtf((float)TILE)};
    // A key-tile step of a two-tile CTA takes ~1.5x that of a one-tile CTA: two tiles per CTA pay off unless they
    // leave SMs empty that one-tile CTAs would fill (short chunks, few heads).
    const int64_t ctas1 = (n + TILE - 1) / TILE * Hq, ctas2 = (n + 2 * TILE - 1) / (2 * TILE) * Hq;
    const int64_t sms = sm_count();
    const bool two = tiles_per_cta == 2 || (tiles_per_cta == 0 && n > TILE && 3 * ((ctas2 + sms - 1) / sms) <= 2 * ((ctas1 + sms - 1) / sms));
    if (two) {
        dim3 grid(Hq, (unsigned)((n + 2 * TILE - 1) / (2 * TILE)));
        SBP_LAUNCH(attn_fwd_2q_kernel, grid, FWD2Q_THREADS, FWD2Q_SMEM, st, mq, mk, mv, p);
        return STREAMBP_OK;
    }
    dim3 grid(Hq, (unsigned)((n + TILE - 1) / TILE));
    SBP_LAUNCH(attn_fwd_tc16_kernel, grid, FWD16_THREADS, FWD16_SMEM, st, mq, mk, mv, p);
    return STREAMBP_OK;
}

int attention_bwd_tc(const bf16 *q, const bf16 *k, const bf16 *v, const bf16 *dout, const float *lse,
                     const float *delta, int64_t n, int64_t q0, int Hq, int Hkv, float *dq, float *dk, float *dv,
                     cudaStream_t st, bool five_products) {
    CUtensorMap mq, mk, mv, mdo;
    const int64_t kv_len = q0 + n;
    if (!make_tensor_map(&mq, q, n, (int64_t)Hq * TILE, (int64_t)Hq * TILE, 64, TILE, false) ||
        !make_tensor_map(&mdo, dout, n, (int64_t)Hq * TILE, (int64_t)Hq * TILE, 64, TILE, false) ||
        !make_tensor_map(&mk, k, kv_len, (int64_t)Hkv * TILE, (int64_t)Hkv * TILE, 64, TILE, false) ||
        !make_tensor_map(&mv, v, kv_len, (int64_t)Hkv * TILE, (int64_t)Hkv * TILE, 64, TILE, false))
        return STREAMBP_E_CUDA;
    static PerDevice configured;
    if (!configured.get([] { return opt_in_smem(attn_bwd_tc_kernel, BWD_FUSED_SMEM) ? 1 : 0; })) return STREAMBP_E_CUDA;
    const float scale = 1.f / sqrtf((float)TILE);
    BwdParams p{(int)n, (long long)q0, Hq, Hkv, lse, delta, dq, dk, dv, scale, scale * kLog2e};
    const int kv_tiles = (int)((kv_len + TILE - 1) / TILE), q_tiles = (int)((n + TILE - 1) / TILE);
    const int64_t n_dkdv = (int64_t)kv_tiles * Hkv, n_dq = (int64_t)q_tiles * Hq;
    if (n_dkdv + n_dq > 0x7fffffff) return STREAMBP_E_SHAPE;
    if (five_products) {
        static PerDevice configured_f;
        if (!configured_f.get([] { return opt_in_smem(attn_bwd_fused_kernel, BWD_SMEM) ? 1 : 0; })) return STREAMBP_E_CUDA;
        CUtensorMap mdq;
        if (!make_tensor_map(&mdq, dq, n, (int64_t)Hq * TILE, (int64_t)Hq * TILE, 32, 32, true)) return STREAMBP_E_CUDA;
        if (!cuda_ok(cudaMemsetAsync(dq, 0, sizeof(float) * (size_t)n * Hq * TILE, st))) return STREAMBP_E_CUDA;
        SBP_LAUNCH(attn_bwd_fused_kernel, (unsigned)n_dkdv, FUSED_THREADS, BWD_SMEM, st, mq, mk, mv, mdo, mdq, p, kv_tiles);
        return STREAMBP_OK;
    }
    // cost of the longest CTA of each role in tile pairs (a dK/dV pair takes ~1.25x a dQ pair: four products against three)
    const int64_t dq_longest = 4 * (int64_t)kv_tiles, dkdv_longest = 5 * (int64_t)(Hq / Hkv) * q_tiles;
    const int n_dq_first = dq_longest > dkdv_longest ? (int)n_dq : 0;
    SBP_LAUNCH(attn_bwd_tc_kernel, (unsigned)(n_dkdv + n_dq), BWD_THREADS, BWD_FUSED_SMEM, st, mq, mk, mv, mdo, p,
               kv_tiles, (int)n_dkdv, q_tiles, n_dq_first);
    return STREAMBP_OK;
}

int attention_tc_take_fault() { return take_fault_local(); }

}  // namespace sbp
