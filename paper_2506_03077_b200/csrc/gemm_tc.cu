// tcgen05 tensor-core GEMM for sm_100a: bf16 operands staged in shared memory by TMA
// (128-byte swizzle), fp32 accumulation in tensor memory, three operand layouts, several
// independent products (each possibly a sum over K segments) per launch.
//
// Two kernels with the same roles, epilogue and tile list:
//   gemm_pair_kernel  : persistent grid of two-CTA clusters (one per TPC), output tile 256 x 256 per pair,
//                       tcgen05.mma.cta_group::2, six 32 KiB operand stages per CTA -- the one that runs
//   gemm_group_kernel : persistent grid, one CTA per SM, output tile 128 x 256, four 48 KiB stages -- the
//                       fallback where a two-CTA cluster cannot be scheduled
// Per CTA, K slices of 64:
//   warp 0      : tile scheduler and TMA producer (one elected lane)
//   warp 1      : allocates tensor memory, issues tcgen05.mma (one elected lane; even CTA of a pair)
//   warps 2..5  : epilogue -- tcgen05.ld of a 32-lane quarter, bias, then
//                 fp32 output: 32x32 blocks staged in shared memory (128-byte swizzle) and written
//                 by TMA store, or added into C by TMA reduce-add when accumulating, so the
//                 read-modify-write of a weight-gradient tile never passes through the SM;
//                 bf16 output: 16-byte stores from registers
//   tensor memory holds two 128 x 256 fp32 accumulators per CTA, so the epilogue of tile i overlaps
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
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "sm100.cuh"

namespace sbp {
namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;   // 16 KiB
constexpr int B_BYTES = BN * BK * 2;   // 32 KiB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int EPI_BUF_BYTES = 32 * 128;                  // one 32 x 32 fp32 block
constexpr int EPI_BYTES = 4 * 2 * EPI_BUF_BYTES;          // 4 epilogue warps, double-buffered
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + 1024 /* alignment slack */ + 256 /* barriers, tile ring */;
constexpr int NUM_THREADS = 192;
constexpr uint32_t TMEM_COLS = 512;
// CTA-pair kernel: a pair works on a 256 x 256 tile, each CTA holding its 128 rows of A and its half of B
constexpr int PAIR_BM = 2 * BM, PAIR_STAGES = 6;
constexpr int PAIR_B_BYTES = (BN / 2) * BK * 2;             // 16 KiB
constexpr int PAIR_STAGE_BYTES = A_BYTES + PAIR_B_BYTES;    // 32 KiB
constexpr int PAIR_SMEM_BYTES = PAIR_STAGES * PAIR_STAGE_BYTES + EPI_BYTES + 1024 + 256;

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
    static PerDevice cache;
    return cache.get([] {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            n = 148;
        return n;
    });
}


namespace {

// ---------------------------------------------------------------------------------------------
// One launch, several products.  A launch carries up to MAX_PROBS independent problems; a problem
// is C (+)= sum over its K segments of op(A_s, B_s), so that e.g. dh2 = dg Wg + du Wu is ONE
// accumulation in tensor memory and not a product followed by a read-modify-write of C.  The tiles
// of all problems form one list, longest tiles first; CTAs take tiles from it either statically
// (tile = blockIdx.x + i * gridDim.x) or, when the caller provides a counter, dynamically with one
// atomicAdd per tile.  Either way an output tile is produced by exactly one CTA in a fixed order of
// K, so results do not depend on the schedule.  Grouping the products that become ready together
// removes most of the part-empty last wave each of them would have on its own.
// Operand layouts, output type and accumulation are per-problem run-time flags.
// ---------------------------------------------------------------------------------------------
constexpr int MAX_PROBS = 4, MAX_SEGS = 8, RING = 4;
constexpr uint32_t F_A_MN = 1u, F_B_MN = 2u, F_OUT_F32 = 4u, F_ACC = 8u, F_SWIGLU = 16u, F_ROPE = 32u;

struct GroupParams {
    CUtensorMap map_a[MAX_SEGS];
    CUtensorMap map_b[MAX_SEGS];
    CUtensorMap map_c[MAX_PROBS];
    int seg_kb[MAX_SEGS];              // K blocks of each segment
    int seg_begin[MAX_PROBS + 1];      // segments of problem q: seg_begin[q] .. seg_begin[q+1]-1
    int tile_begin[MAX_PROBS + 1];     // tiles of problem q: tile_begin[q] .. tile_begin[q+1]-1
    int tiles_m[MAX_PROBS];
    int M[MAX_PROBS], N[MAX_PROBS];
    void *C[MAX_PROBS];
    void *C_up[MAX_PROBS], *C_act[MAX_PROBS];   // SwiGLU pairs: u and silu(g) * u beside g in C
    long long ldc[MAX_PROBS];
    const bf16 *bias[MAX_PROBS];
    const float2 *rope[MAX_PROBS];     // F_ROPE: (cos, sin) of 64 frequencies per row of the problem
    uint32_t flags[MAX_PROBS];
    int nprob;
    int *sched;                        // {next tile, CTAs finished}, both zero at launch; or nullptr: static schedule
    const int *gate;                   // optional: the kernel returns at once when *gate == 0
};

template <typename T>
__device__ __forceinline__ T pick(const T (&a)[MAX_PROBS], int q) {
    T v = a[0];
#pragma unroll
    for (int i = 1; i < MAX_PROBS; i++) v = (q == i) ? a[i] : v;
    return v;
}

struct TileRef { int q, m0, n0, seg0, seg1; };
template <int TILE_M>
__device__ __forceinline__ TileRef locate(const GroupParams &p, int tile) {
    int q = 0;
#pragma unroll
    for (int i = 1; i < MAX_PROBS; i++) q = (i < p.nprob && tile >= p.tile_begin[i]) ? i : q;
    int tb = p.tile_begin[0], s0 = p.seg_begin[0], s1 = p.seg_begin[1];
#pragma unroll
    for (int i = 1; i < MAX_PROBS; i++) {
        tb = (q == i) ? p.tile_begin[i] : tb;
        s0 = (q == i) ? p.seg_begin[i] : s0;
        s1 = (q == i) ? p.seg_begin[i + 1] : s1;
    }
    const int local = tile - tb, tm = pick(p.tiles_m, q);
    // a SwiGLU pair has two B operands (W_gate, W_up: segments s0, s0 + 1) but ONE pass over K
    if (pick(p.flags, q) & F_SWIGLU) s1 = s0 + 1;
    return {q, (local % tm) * TILE_M, (local / tm) * BN, s0, s1};
}

// The K loops of one tile, specialised on the operand layouts so that descriptor strides and the choice of
// TMA boxes are compile-time constants (a run-time layout costs ~10 % on MN-major operands: the two
// single-thread issue paths are the critical ones).
struct Pipe {
    uint32_t tiles, bar_full, bar_empty;
    volatile int *abort_flag;
};

template <bool A_MN, bool B_MN>
__device__ __forceinline__ bool produce_tile(const GroupParams &p, const TileRef &t, const Pipe &pp, uint32_t &stage,
                                             uint32_t &phase) {
    for (int s = t.seg0; s < t.seg1; s++) {
        const CUtensorMap *ma = &p.map_a[s], *mb = &p.map_b[s];
        const int nkb = p.seg_kb[s];
        for (int kb = 0; kb < nkb; kb++) {
            if (!mbar_wait(pp.bar_empty + 8 * stage, phase ^ 1u, pp.abort_flag)) return false;
            const uint32_t full = pp.bar_full + 8 * stage;
            const uint32_t sa = pp.tiles + stage * STAGE_BYTES, sb = sa + A_BYTES;
            mbar_expect_tx(full, STAGE_BYTES);
            const int k0 = kb * BK;
            if (A_MN) {
#pragma unroll
                for (int j = 0; j < BM / 64; j++) tma_load_2d(sa + j * 8192, ma, full, t.m0 + 64 * j, k0);
            } else {
                tma_load_2d(sa, ma, full, k0, t.m0);
            }
            if (B_MN) {
#pragma unroll
                for (int j = 0; j < BN / 64; j++) tma_load_2d(sb + j * 8192, mb, full, t.n0 + 64 * j, k0);
            } else {
                tma_load_2d(sb, mb, full, k0, t.n0);
            }
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
    }
    return true;
}

template <bool A_MN, bool B_MN>
__device__ __forceinline__ bool mma_tile(const GroupParams &p, const TileRef &t, const Pipe &pp, uint32_t d_tmem,
                                         uint32_t &stage, uint32_t &phase) {
    constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) |
                               ((B_MN ? 1u : 0u) << 16) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
    constexpr uint32_t a_step = A_MN ? 2048u : 32u, b_step = B_MN ? 2048u : 32u;   // bytes per 16 k
    uint32_t first = 0;
    for (int s = t.seg0; s < t.seg1; s++) {
        const int nkb = p.seg_kb[s];
        for (int kb = 0; kb < nkb; kb++) {
            if (!mbar_wait(pp.bar_full + 8 * stage, phase, pp.abort_flag)) return false;
            tc_fence_after();
            const uint32_t sa = pp.tiles + stage * STAGE_BYTES, sb = sa + A_BYTES;
            const uint32_t a_lo = desc_lo(sa, A_MN ? 8192u : 16u), b_lo = desc_lo(sb, B_MN ? 8192u : 16u);
#pragma unroll
            for (int kk = 0; kk < BK / 16; kk++)
                umma_ss(d_tmem, a_lo + kk * (a_step >> 4), b_lo + kk * (b_step >> 4), idesc, first | (uint32_t)kk);
            first = 1u;
            umma_commit(pp.bar_empty + 8 * stage);   // frees the stage once these MMAs have read it
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
    }
    return true;
}

// One epilogue warp: rows m_base + 32 * quarter .. + 31 of tile t, all BN columns, from the accumulator at `acc`
// (lane = row).  fp32 output: 32 x 32 blocks staged in shared memory with the 128-byte swizzle the tensor map expects,
// then a TMA store, or a TMA reduce-add when accumulating; bf16 output: 16-byte stores from registers.
__device__ __forceinline__ void epilogue_rows(const GroupParams &p, const TileRef &t, int m_base, int quarter, int lane,
                                              uint32_t acc, uint32_t epi, uint32_t &staged) {
    const uint32_t fl = pick(p.flags, t.q);
    const int Mq = pick(p.M, t.q), Nq = pick(p.N, t.q);
    const bf16 *bias = pick(p.bias, t.q);
    const CUtensorMap *mc = &p.map_c[t.q];
    const int row = m_base + quarter * 32 + lane;
    const uint32_t taddr = acc + ((uint32_t)(quarter * 32) << 16);
    if (fl & F_SWIGLU) {
        // accumulator columns c and 128 + c are g and u of output column n0 / 2 + c: round both to bf16 (what the
        // backward will read), m = silu(g) * u from the rounded values, three 16-byte stores per 8 columns
        const long long off = (long long)row * pick(p.ldc, t.q);
        bf16 *og = reinterpret_cast<bf16 *>(pick(p.C, t.q)) + off, *ou = reinterpret_cast<bf16 *>(pick(p.C_up, t.q)) + off,
             *om = reinterpret_cast<bf16 *>(pick(p.C_act, t.q)) + off;
#pragma unroll 1
        for (int c = 0; c < BN / 64; c++) {
            const int col0 = t.n0 / 2 + c * 32;
            if (col0 >= Nq) break;               // uniform across the warp
            uint32_t rg[32], ru[32];
            tmem_ld32(taddr + c * 32, rg);
            tmem_ld32(taddr + BN / 2 + c * 32, ru);
            if (row >= Mq) continue;
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
                uint32_t wg[4], wu[4], wm[4];
#pragma unroll
                for (int e = 0; e < 4; e++) {
                    const __nv_bfloat162 hg = __floats2bfloat162_rn(__uint_as_float(rg[j + 2 * e]), __uint_as_float(rg[j + 2 * e + 1]));
                    const __nv_bfloat162 hu = __floats2bfloat162_rn(__uint_as_float(ru[j + 2 * e]), __uint_as_float(ru[j + 2 * e + 1]));
                    const float2 fg = __bfloat1622float2(hg), fu = __bfloat1622float2(hu);
                    const float m0 = fg.x * (1.f / (1.f + __expf(-fg.x))) * fu.x;
                    const float m1 = fg.y * (1.f / (1.f + __expf(-fg.y))) * fu.y;
                    const __nv_bfloat162 hm = __floats2bfloat162_rn(m0, m1);
                    wg[e] = *reinterpret_cast<const uint32_t *>(&hg);
                    wu[e] = *reinterpret_cast<const uint32_t *>(&hu);
                    wm[e] = *reinterpret_cast<const uint32_t *>(&hm);
                }
                if (col0 + j + 7 < Nq) {
                    *reinterpret_cast<uint4 *>(og + col0 + j) = make_uint4(wg[0], wg[1], wg[2], wg[3]);
                    *reinterpret_cast<uint4 *>(ou + col0 + j) = make_uint4(wu[0], wu[1], wu[2], wu[3]);
                    *reinterpret_cast<uint4 *>(om + col0 + j) = make_uint4(wm[0], wm[1], wm[2], wm[3]);
                } else {
                    const bf16 *sg = reinterpret_cast<const bf16 *>(wg), *su = reinterpret_cast<const bf16 *>(wu),
                               *sm = reinterpret_cast<const bf16 *>(wm);
                    for (int e = 0; e < 8; e++)
                        if (col0 + j + e < Nq) {
                            og[col0 + j + e] = sg[e];
                            ou[col0 + j + e] = su[e];
                            om[col0 + j + e] = sm[e];
                        }
                }
            }
        }
        return;
    }
    bf16 *out_row = reinterpret_cast<bf16 *>(pick(p.C, t.q)) + (long long)row * pick(p.ldc, t.q);
    if (fl & F_ROPE) {
        // rotary embedding of 128-wide heads (a tile holds two): the accumulator columns of a head are [x1 | x2],
        // 64 each; out1 = x1 cos - x2 sin, out2 = x2 cos + x1 sin with the row's (cos, sin) of frequency j, in fp32
        // from the accumulator (+ bias), rounded to bf16 once.  N is a multiple of 128 (checked on the host).
        const float2 *cs = pick(p.rope, t.q) + (long long)(row < Mq ? row : 0) * 64;
#pragma unroll 1
        for (int f0 = 0; f0 < 64; f0 += 32) {
            // the row's (cos, sin) of 32 frequencies, fetched once for both heads of the tile
            float4 q[16];
#pragma unroll
            for (int e = 0; e < 16; e++) q[e] = *reinterpret_cast<const float4 *>(cs + f0 + 2 * e);
#pragma unroll 1
            for (int head = 0; head < BN / 128; head++) {
                const int col0 = t.n0 + head * 128;
                if (col0 >= Nq) break;               // uniform across the warp
                uint32_t ra[32], rb[32];
                tmem_ld32(taddr + head * 128 + f0, ra);
                tmem_ld32(taddr + head * 128 + 64 + f0, rb);
                if (row >= Mq) continue;
#pragma unroll
                for (int j = 0; j < 32; j += 8) {
                    uint32_t w1[4], w2[4];
#pragma unroll
                    for (int e = 0; e < 4; e++) {
                        float a0 = __uint_as_float(ra[j + 2 * e]), a1 = __uint_as_float(ra[j + 2 * e + 1]);
                        float b0 = __uint_as_float(rb[j + 2 * e]), b1 = __uint_as_float(rb[j + 2 * e + 1]);
                        if (bias) {
                            const __nv_bfloat162 ba = *reinterpret_cast<const __nv_bfloat162 *>(bias + col0 + f0 + j + 2 * e);
                            const __nv_bfloat162 bb = *reinterpret_cast<const __nv_bfloat162 *>(bias + col0 + 64 + f0 + j + 2 * e);
                            a0 += __low2float(ba); a1 += __high2float(ba);
                            b0 += __low2float(bb); b1 += __high2float(bb);
                        }
                        const float4 k = q[(j >> 1) + e];       // (cos, sin) of frequencies f0 + j + 2e, + 1
                        const __nv_bfloat162 h1 = __floats2bfloat162_rn(a0 * k.x - b0 * k.y, a1 * k.z - b1 * k.w);
                        const __nv_bfloat162 h2 = __floats2bfloat162_rn(b0 * k.x + a0 * k.y, b1 * k.z + a1 * k.w);
                        w1[e] = *reinterpret_cast<const uint32_t *>(&h1);
                        w2[e] = *reinterpret_cast<const uint32_t *>(&h2);
                    }
                    *reinterpret_cast<uint4 *>(out_row + col0 + f0 + j) = make_uint4(w1[0], w1[1], w1[2], w1[3]);
                    *reinterpret_cast<uint4 *>(out_row + col0 + 64 + f0 + j) = make_uint4(w2[0], w2[1], w2[2], w2[3]);
                }
            }
        }
        return;
    }
#pragma unroll 1
    for (int c = 0; c < BN / 32; c++) {
        const int col0 = t.n0 + c * 32;
        if (col0 >= Nq) break;               // uniform across the warp
        uint32_t r[32];
        tmem_ld32(taddr + c * 32, r);
        if (fl & F_OUT_F32) {
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
                    if (bias && col0 + 4 * j + e < Nq) v[e] += __bfloat162float(bias[col0 + 4 * j + e]);
                }
                const uint32_t dst = buf_s + lane * 128 + ((j ^ (lane & 7)) << 4);
                asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(v[0]), "f"(v[1]),
                             "f"(v[2]), "f"(v[3])
                             : "memory");
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                if (fl & F_ACC) tma_reduce_add_2d(mc, buf_s, col0, m_base + quarter * 32);
                else tma_store_2d(mc, buf_s, col0, m_base + quarter * 32);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
        } else if (row < Mq) {
            bf16 *out = out_row + col0;
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
                float v[8];
#pragma unroll
                for (int e = 0; e < 8; e++) {
                    v[e] = __uint_as_float(r[j + e]);
                    if (bias && col0 + j + e < Nq) v[e] += __bfloat162float(bias[col0 + j + e]);
                }
                if (col0 + j + 7 < Nq) {
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; e++) {
                        __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
                        w[e] = *reinterpret_cast<uint32_t *>(&h);
                    }
                    *reinterpret_cast<uint4 *>(out + j) = make_uint4(w[0], w[1], w[2], w[3]);
                } else {
                    for (int e = 0; e < 8; e++)
                        if (col0 + j + e < Nq) out[j + e] = __float2bfloat16_rn(v[e]);
                }
            }
        }
    }
}

__global__ void __launch_bounds__(NUM_THREADS, 1) gemm_group_kernel(const __grid_constant__ GroupParams p) {
    pdl_enter();
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
    const uint32_t bar_rfull = bar_tempty + 16;              // RING x 8 B: a tile index has been published
    const uint32_t bar_rempty = bar_rfull + 8 * RING;        // RING x 8 B: all five readers have taken it
    uint8_t *aux2 = aux + 8 * STAGES * 2 + 32 + 16 * RING;
    volatile int *ring = reinterpret_cast<volatile int *>(aux2);              // RING tile indices
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(aux2 + 4 * RING);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(aux2 + 4 * RING + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_tiles = p.tile_begin[p.nprob < MAX_PROBS ? p.nprob : MAX_PROBS];

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; s++) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; b++) {
            mbar_init(bar_tfull + 8 * b, 1);
            mbar_init(bar_tempty + 8 * b, 4);
        }
        for (int s = 0; s < RING; s++) {
            mbar_init(bar_rfull + 8 * s, 1);
            mbar_init(bar_rempty + 8 * s, 5);       // MMA thread + four epilogue warps
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------ tile scheduler + TMA producer ------------------------------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, slot = 0, rphase = 0;
            const bool dynamic = p.sched != nullptr;
            int tile = dynamic ? atomicAdd(p.sched, 1) : (int)blockIdx.x;
            bool alive = true;
            while (alive) {
                if (tile >= num_tiles) tile = -1;
                if (!mbar_wait(bar_rempty + 8 * slot, rphase ^ 1u, abort_flag)) break;
                ring[slot] = tile;
                mbar_arrive(bar_rfull + 8 * slot);
                if (++slot == RING) { slot = 0; rphase ^= 1u; }
                if (tile < 0) break;
                // the next index is requested now and first looked at after this tile's loads are issued
                const int next = dynamic ? atomicAdd(p.sched, 1) : tile + (int)gridDim.x;
                const TileRef t = locate<BM>(p, tile);
                const uint32_t fl = pick(p.flags, t.q);
                const Pipe pipe{tiles, bar_full, bar_empty, abort_flag};
                switch (fl & (F_A_MN | F_B_MN)) {
                    case 0: alive = produce_tile<false, false>(p, t, pipe, stage, phase); break;
                    case F_B_MN: alive = produce_tile<false, true>(p, t, pipe, stage, phase); break;
                    default: alive = produce_tile<true, true>(p, t, pipe, stage, phase); break;
                }
                tile = next;
            }
            if (dynamic) {
                // every CTA takes exactly one index past the end; the last CTA to get there re-arms the counter
                __threadfence();
                if (atomicAdd(p.sched + 1, 1) == (int)gridDim.x - 1) {
                    p.sched[0] = 0;
                    p.sched[1] = 0;
                    __threadfence();
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, slot = 0, rphase = 0, local = 0;
            bool alive = true;
            while (alive) {
                if (!mbar_wait(bar_rfull + 8 * slot, rphase, abort_flag)) break;
                const int tile = ring[slot];
                mbar_arrive(bar_rempty + 8 * slot);
                if (++slot == RING) { slot = 0; rphase ^= 1u; }
                if (tile < 0) break;
                const TileRef t = locate<BM>(p, tile);
                const uint32_t fl = pick(p.flags, t.q);
                const uint32_t buf = local & 1u, use = local >> 1;
                if (!mbar_wait(bar_tempty + 8 * buf, (use & 1u) ^ 1u, abort_flag)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                const Pipe pipe{tiles, bar_full, bar_empty, abort_flag};
                switch (fl & (F_A_MN | F_B_MN)) {
                    case 0: alive = mma_tile<false, false>(p, t, pipe, d_tmem, stage, phase); break;
                    case F_B_MN: alive = mma_tile<false, true>(p, t, pipe, d_tmem, stage, phase); break;
                    default: alive = mma_tile<true, true>(p, t, pipe, d_tmem, stage, phase); break;
                }
                if (alive) umma_commit(bar_tfull + 8 * buf);   // accumulator complete
                local++;
            }
        }
    } else {
        // ------------------------------ epilogue ------------------------------
        const int quarter = warp & 3;                 // TMEM lanes 32*quarter .. +31
        uint32_t local = 0, staged = 0, slot = 0, rphase = 0;   // staged: fp32 blocks this warp has sent so far
        while (true) {
            if (!mbar_wait(bar_rfull + 8 * slot, rphase, abort_flag)) break;
            const int tile = ring[slot];
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_rempty + 8 * slot);
            if (++slot == RING) { slot = 0; rphase ^= 1u; }
            if (tile < 0) break;
            const TileRef t = locate<BM>(p, tile);
            const uint32_t buf = local & 1u, use = local >> 1;
            local++;
            if (!mbar_wait(bar_tfull + 8 * buf, use & 1u, abort_flag)) break;
            tc_fence_after();
            epilogue_rows(p, t, t.m0, quarter, lane, tmem_base + buf * BN, epi, staged);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
        }
    }

    if (warp >= 2 && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
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
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ---------------------------------------------------------------------------------------------
// CTA-pair variant (tcgen05 cta_group::2).  The two CTAs of a cluster sit on the two SMs of one TPC and
// share every MMA: a 256 x 256 x 64 step is issued by the even CTA, reads 128 rows of A and 128 rows of B
// from the shared memory of EACH CTA and leaves 128 rows of the accumulator in the tensor memory of each.
// Per CTA a K slice is then 32 KiB instead of 48, so the same shared memory holds six stages instead of
// four -- the main loop of the single-CTA kernel spends about half of its time waiting for operand copies
// (their latency under load is ~3000 cycles, four 512-cycle slices do not cover it) -- and a third less
// data crosses L2 -> SM per FLOP.  Roles per CTA as in gemm_group_kernel; in addition
//   * the even CTA's scheduler thread publishes each tile index in both CTAs' rings,
//   * operand copies of both CTAs report to the even CTA's `full` barrier (armed there with the bytes of
//     both); the MMA thread's commits arrive at `empty` / `tfull` in both CTAs,
//   * the odd CTA's ring readers and epilogue warps arrive at the even CTA's `rempty` / `tempty`.
// No copy is multicast: each CTA fetches its own operand rows.
// ---------------------------------------------------------------------------------------------
template <bool A_MN, bool B_MN>
__device__ __forceinline__ bool produce_tile_pair(const GroupParams &p, const TileRef &t, const Pipe &pp, uint32_t rank,
                                                  uint32_t &stage, uint32_t &phase) {
    // SwiGLU pair: both CTAs fetch the SAME 128 weight rows, the even one of W_gate, the odd one of W_up, so that
    // accumulator columns 0..127 hold g and 128..255 hold u of output columns n0 / 2 ..
    const bool swiglu = (pick(p.flags, t.q) & F_SWIGLU) != 0;
    const int m = t.m0 + BM * (int)rank, n = swiglu ? t.n0 / 2 : t.n0 + (BN / 2) * (int)rank;
    for (int s = t.seg0; s < t.seg1; s++) {
        const CUtensorMap *ma = &p.map_a[s], *mb = &p.map_b[s + ((swiglu && rank) ? 1 : 0)];
        const int nkb = p.seg_kb[s];
        for (int kb = 0; kb < nkb; kb++) {
            if (!mbar_wait(pp.bar_empty + 8 * stage, phase ^ 1u, pp.abort_flag)) return false;
            if (rank == 0) mbar_expect_tx(pp.bar_full + 8 * stage, 2 * PAIR_STAGE_BYTES);
            const uint32_t full = map_to_cta(pp.bar_full + 8 * stage, 0);
            const uint32_t sa = pp.tiles + stage * PAIR_STAGE_BYTES, sb = sa + A_BYTES;
            const int k0 = kb * BK;
            if (A_MN) {
#pragma unroll
                for (int j = 0; j < BM / 64; j++) tma_load_2d_pair(sa + j * 8192, ma, full, m + 64 * j, k0);
            } else {
                tma_load_2d_pair(sa, ma, full, k0, m);
            }
            if (B_MN) {
#pragma unroll
                for (int j = 0; j < BN / 128; j++) tma_load_2d_pair(sb + j * 8192, mb, full, n + 64 * j, k0);
            } else {
                tma_load_2d_pair(sb, mb, full, k0, n);
            }
            if (++stage == PAIR_STAGES) { stage = 0; phase ^= 1u; }
        }
    }
    return true;
}

template <bool A_MN, bool B_MN>
__device__ __forceinline__ bool mma_tile_pair(const GroupParams &p, const TileRef &t, const Pipe &pp, uint32_t d_tmem,
                                              uint32_t &stage, uint32_t &phase) {
    constexpr uint32_t idesc = make_idesc(PAIR_BM, BN, A_MN, B_MN);
    constexpr uint32_t a_step = A_MN ? 2048u : 32u, b_step = B_MN ? 2048u : 32u;   // bytes per 16 k
    uint32_t first = 0;
    for (int s = t.seg0; s < t.seg1; s++) {
        const int nkb = p.seg_kb[s];
        for (int kb = 0; kb < nkb; kb++) {
            if (!mbar_wait_cluster(pp.bar_full + 8 * stage, phase, pp.abort_flag)) return false;
            tc_fence_after();
            const uint32_t sa = pp.tiles + stage * PAIR_STAGE_BYTES, sb = sa + A_BYTES;
            const uint32_t a_lo = desc_lo(sa, A_MN ? 8192u : 16u), b_lo = desc_lo(sb, B_MN ? 8192u : 16u);
#pragma unroll
            for (int kk = 0; kk < BK / 16; kk++)
                umma_ss_pair(d_tmem, a_lo + kk * (a_step >> 4), b_lo + kk * (b_step >> 4), idesc, first | (uint32_t)kk);
            first = 1u;
            umma_commit_pair(pp.bar_empty + 8 * stage);   // frees the stage in both CTAs
            if (++stage == PAIR_STAGES) { stage = 0; phase ^= 1u; }
        }
    }
    return true;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
    gemm_pair_kernel(const __grid_constant__ GroupParams p) {
    pdl_enter();
    extern __shared__ uint8_t smem_raw[];
    if (gated_off(p.gate)) return;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    const uint32_t epi = tiles + PAIR_STAGES * PAIR_STAGE_BYTES;
    uint8_t *aux = smem_raw + (tiles - raw) + PAIR_STAGES * PAIR_STAGE_BYTES + EPI_BYTES;
    const uint32_t bar_full = smem_u32(aux);                  // PAIR_STAGES x 8 B, used in the even CTA
    const uint32_t bar_empty = bar_full + 8 * PAIR_STAGES;    // PAIR_STAGES x 8 B, in both
    const uint32_t bar_tfull = bar_empty + 8 * PAIR_STAGES;   // 2 x 8 B, in both
    const uint32_t bar_tempty = bar_tfull + 16;               // 2 x 8 B, even CTA: eight epilogue warps arrive
    const uint32_t bar_rfull = bar_tempty + 16;               // RING x 8 B, in both
    const uint32_t bar_rempty = bar_rfull + 8 * RING;         // RING x 8 B, even CTA: ten readers arrive
    uint8_t *aux2 = aux + 8 * PAIR_STAGES * 2 + 32 + 16 * RING;
    volatile int *ring = reinterpret_cast<volatile int *>(aux2);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(aux2 + 4 * RING);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(aux2 + 4 * RING + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_cta_rank();
    const int num_tiles = p.tile_begin[p.nprob < MAX_PROBS ? p.nprob : MAX_PROBS];

    if (threadIdx.x == 0) {
        for (int s = 0; s < PAIR_STAGES; s++) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; b++) {
            mbar_init(bar_tfull + 8 * b, 1);
            mbar_init(bar_tempty + 8 * b, 8);
        }
        for (int s = 0; s < RING; s++) {
            mbar_init(bar_rfull + 8 * s, 1);
            mbar_init(bar_rempty + 8 * s, 10);      // even CTA: MMA thread + 4 epilogue warps; odd CTA: producer + 4
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();            // both CTAs' barriers exist before anything arrives at them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const Pipe pipe{tiles, bar_full, bar_empty, abort_flag};

    if (warp == 0) {
        // ------------------------------ tile scheduler (even CTA) + TMA producer ------------------------------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, slot = 0, rphase = 0;
            bool alive = true;
            if (rank == 0) {
                const bool dynamic = p.sched != nullptr;
                const int npairs = (int)(gridDim.x >> 1);
                int tile = dynamic ? atomicAdd(p.sched, 1) : (int)(blockIdx.x >> 1);
                while (alive) {
                    if (tile >= num_tiles) tile = -1;
                    if (!mbar_wait_cluster(bar_rempty + 8 * slot, rphase ^ 1u, abort_flag)) break;
                    ring[slot] = tile;
                    st_remote_u32(map_to_cta(smem_u32(const_cast<int *>(ring + slot)), 1), (uint32_t)tile);
                    mbar_arrive(bar_rfull + 8 * slot);
                    mbar_arrive_remote(map_to_cta(bar_rfull + 8 * slot, 1));
                    if (++slot == RING) { slot = 0; rphase ^= 1u; }
                    if (tile < 0) break;
                    const int next = dynamic ? atomicAdd(p.sched, 1) : tile + npairs;
                    const TileRef t = locate<PAIR_BM>(p, tile);
                    switch (pick(p.flags, t.q) & (F_A_MN | F_B_MN)) {
                        case 0: alive = produce_tile_pair<false, false>(p, t, pipe, 0u, stage, phase); break;
                        case F_B_MN: alive = produce_tile_pair<false, true>(p, t, pipe, 0u, stage, phase); break;
                        default: alive = produce_tile_pair<true, true>(p, t, pipe, 0u, stage, phase); break;
                    }
                    tile = next;
                }
                if (dynamic) {
                    // every pair takes exactly one index past the end; the last one to get there re-arms the counter
                    __threadfence();
                    if (atomicAdd(p.sched + 1, 1) == npairs - 1) {
                        p.sched[0] = 0;
                        p.sched[1] = 0;
                        __threadfence();
                    }
                }
            } else {
                while (alive) {
                    if (!mbar_wait_cluster(bar_rfull + 8 * slot, rphase, abort_flag)) break;
                    const int tile = ring[slot];
                    mbar_arrive_remote(map_to_cta(bar_rempty + 8 * slot, 0));
                    if (++slot == RING) { slot = 0; rphase ^= 1u; }
                    if (tile < 0) break;
                    const TileRef t = locate<PAIR_BM>(p, tile);
                    switch (pick(p.flags, t.q) & (F_A_MN | F_B_MN)) {
                        case 0: alive = produce_tile_pair<false, false>(p, t, pipe, 1u, stage, phase); break;
                        case F_B_MN: alive = produce_tile_pair<false, true>(p, t, pipe, 1u, stage, phase); break;
                        default: alive = produce_tile_pair<true, true>(p, t, pipe, 1u, stage, phase); break;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer (even CTA only) ------------------------------
        if (lane == 0 && rank == 0) {
            uint32_t stage = 0, phase = 0, slot = 0, rphase = 0, local = 0;
            bool alive = true;
            while (alive) {
                if (!mbar_wait(bar_rfull + 8 * slot, rphase, abort_flag)) break;
                const int tile = ring[slot];
                mbar_arrive(bar_rempty + 8 * slot);
                if (++slot == RING) { slot = 0; rphase ^= 1u; }
                if (tile < 0) break;
                const TileRef t = locate<PAIR_BM>(p, tile);
                const uint32_t buf = local & 1u, use = local >> 1;
                if (!mbar_wait_cluster(bar_tempty + 8 * buf, (use & 1u) ^ 1u, abort_flag)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                switch (pick(p.flags, t.q) & (F_A_MN | F_B_MN)) {
                    case 0: alive = mma_tile_pair<false, false>(p, t, pipe, d_tmem, stage, phase); break;
                    case F_B_MN: alive = mma_tile_pair<false, true>(p, t, pipe, d_tmem, stage, phase); break;
                    default: alive = mma_tile_pair<true, true>(p, t, pipe, d_tmem, stage, phase); break;
                }
                if (alive) umma_commit_pair(bar_tfull + 8 * buf);   // accumulator complete, in both CTAs
                local++;
            }
        }
    } else {
        // ------------------------------ epilogue: this CTA's 128 rows of the tile ------------------------------
        const int quarter = warp & 3;
        uint32_t local = 0, staged = 0, slot = 0, rphase = 0;
        while (true) {
            if (!mbar_wait_cluster(bar_rfull + 8 * slot, rphase, abort_flag)) break;
            const int tile = ring[slot];
            __syncwarp();
            if (lane == 0) {
                if (rank == 0) mbar_arrive(bar_rempty + 8 * slot);
                else mbar_arrive_remote(map_to_cta(bar_rempty + 8 * slot, 0));
            }
            if (++slot == RING) { slot = 0; rphase ^= 1u; }
            if (tile < 0) break;
            const TileRef t = locate<PAIR_BM>(p, tile);
            const uint32_t buf = local & 1u, use = local >> 1;
            local++;
            if (!mbar_wait(bar_tfull + 8 * buf, use & 1u, abort_flag)) break;
            tc_fence_after();
            epilogue_rows(p, t, t.m0 + BM * (int)rank, quarter, lane, tmem_base + buf * BN, epi, staged);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (rank == 0) mbar_arrive(bar_tempty + 8 * buf);
                else mbar_arrive_remote(map_to_cta(bar_tempty + 8 * buf, 0));
            }
        }
    }

    if (warp >= 2 && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    __syncwarp();
    if (*abort_flag) {
        const unsigned long long t0 = global_timer();
        while (global_timer() - t0 < 200000ull) { }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();            // neither CTA's shared or tensor memory goes away while the other may still reach it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
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

namespace {
// The CTA-pair kernel needs clusters of two CTAs with the full shared-memory carve-out; where the device cannot
// co-schedule even one such cluster the single-CTA kernel runs instead.
bool pair_kernel_available() {
    static PerDevice cache;
    return cache.get([] {
        int state = 0;
        if (cudaFuncSetAttribute(gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PAIR_SMEM_BYTES) ==
            cudaSuccess) {
            cudaLaunchConfig_t cfg;
            memset(&cfg, 0, sizeof(cfg));
            cfg.gridDim = dim3(2, 1, 1);
            cfg.blockDim = dim3(NUM_THREADS, 1, 1);
            cfg.dynamicSmemBytes = PAIR_SMEM_BYTES;
            int clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&clusters, gemm_pair_kernel, &cfg) == cudaSuccess && clusters >= 1)
                state = 1;
        }
        cudaGetLastError();
        if (getenv("STREAMBP_GEMM_SINGLE_CTA")) state = 0;
        if (getenv("STREAMBP_VERBOSE")) fprintf(stderr, "streambp: tcgen05 product kernel: %s\n", state ? "CTA pairs" : "single CTA");
        return state;
    }) == 1;
}
}  // namespace

bool gemm_tc_group_supported(const GemmProb *probs, int n) {
    if (n < 1 || n > MAX_PROBS) return false;
    int segs = 0;
    for (int i = 0; i < n; i++) {
        const GemmProb &g = probs[i];
        if (g.nseg < 1 || g.nseg > 3) return false;
        if (!g.c_is_f32 && g.accumulate) return false;
        if (g.swiglu) {
            auto al16 = [](const void *q) { return q != nullptr && (reinterpret_cast<uintptr_t>(q) & 15u) == 0; };
            if (g.op != OP_NT || g.nseg != 2 || g.c_is_f32 || g.accumulate || g.bias || g.seg[0].K != g.seg[1].K ||
                !al16(g.C_up) || !al16(g.C_act) || !pair_kernel_available())
                return false;
        }
        if (g.rope && (g.c_is_f32 || g.accumulate || g.swiglu || (g.N % 128) ||
                       (reinterpret_cast<uintptr_t>(g.rope) & 15u)))
            return false;
        segs += g.nseg;
        for (int s = 0; s < g.nseg; s++)
            if (!gemm_tc_supported(g.op, g.M, g.N, g.seg[s].K, g.seg[s].lda, g.seg[s].ldb, g.ldc, g.seg[s].A,
                                   g.seg[s].B, g.C, g.c_is_f32))
                return false;
    }
    return segs <= MAX_SEGS;
}


int gemm_tc_group(const GemmProb *probs, int n, int *sched, cudaStream_t st) {
    if (!gemm_tc_group_supported(probs, n)) return STREAMBP_E_SHAPE;
    const bool pair = pair_kernel_available();
    const int tile_m = pair ? PAIR_BM : BM;
    // longest tiles first: with a dynamic schedule the short tiles then fill the gaps the long ones leave
    int order[MAX_PROBS];
    int64_t cost[MAX_PROBS];
    for (int i = 0; i < n; i++) {
        order[i] = i;
        cost[i] = 0;
        for (int s = 0; s < (probs[i].swiglu ? 1 : probs[i].nseg); s++) cost[i] += (probs[i].seg[s].K + BK - 1) / BK;
    }
    for (int i = 1; i < n; i++)
        for (int j = i; j > 0 && cost[order[j]] > cost[order[j - 1]]; j--) {
            const int t = order[j]; order[j] = order[j - 1]; order[j - 1] = t;
        }
    GroupParams p;
    memset(&p, 0, sizeof(p));
    p.nprob = n;
    int seg = 0;
    int64_t tiles = 0;
    for (int i = 0; i < n; i++) {
        const GemmProb &g = probs[order[i]];
        p.seg_begin[i] = seg;
        p.tile_begin[i] = (int)tiles;
        const bool a_mn = g.op == OP_TN, b_mn = g.op != OP_NT;
        for (int s = 0; s < g.nseg; s++, seg++) {
            const GemmSeg &e = g.seg[s];
            bool ok;
            // K-major operands: [rows][64 k] boxes; MN-major operands: [64 k][64 mn] boxes
            if (a_mn) ok = make_tensor_map(&p.map_a[seg], e.A, e.K, g.M, e.lda, 64, BK, false);
            else ok = make_tensor_map(&p.map_a[seg], e.A, g.M, e.K, e.lda, BK, BM, false);
            if (b_mn) ok = ok && make_tensor_map(&p.map_b[seg], e.B, e.K, g.N, e.ldb, 64, BK, false);
            else ok = ok && make_tensor_map(&p.map_b[seg], e.B, g.N, e.K, e.ldb, BK, pair ? BN / 2 : BN, false);
            if (!ok) return STREAMBP_E_CUDA;
            p.seg_kb[seg] = (int)((e.K + BK - 1) / BK);
        }
        if (g.c_is_f32) {
            if (!make_tensor_map(&p.map_c[i], g.C, g.M, g.N, g.ldc, 32, 32, true)) return STREAMBP_E_CUDA;
        } else {
            p.map_c[i] = p.map_a[p.seg_begin[i]];   // unused by bf16 outputs
        }
        p.tiles_m[i] = (int)((g.M + tile_m - 1) / tile_m);
        p.M[i] = (int)g.M;
        p.N[i] = (int)g.N;
        p.C[i] = g.C;
        p.ldc[i] = g.ldc;
        p.bias[i] = g.bias;
        p.rope[i] = reinterpret_cast<const float2 *>(g.rope);
        p.C_up[i] = g.C_up;
        p.C_act[i] = g.C_act;
        p.flags[i] = (a_mn ? F_A_MN : 0u) | (b_mn ? F_B_MN : 0u) | (g.c_is_f32 ? F_OUT_F32 : 0u) |
                     (g.accumulate ? F_ACC : 0u) | (g.swiglu ? F_SWIGLU : 0u) | (g.rope ? F_ROPE : 0u);
        // a SwiGLU tile covers BN / 2 output columns (g and u of the same columns side by side in the accumulator)
        const int64_t tile_n = g.swiglu ? BN / 2 : BN;
        tiles += (int64_t)p.tiles_m[i] * ((g.N + tile_n - 1) / tile_n);
        if (tiles > (1ll << 30)) return STREAMBP_E_SHAPE;
    }
    for (int i = n; i <= MAX_PROBS; i++) {
        p.seg_begin[i] = seg;
        p.tile_begin[i] = (int)tiles;
    }
    p.sched = sched;
    p.gate = call_state().gate;
    static PerDevice configured;
    if (!configured.get([] {
            return cuda_ok(cudaFuncSetAttribute(gemm_group_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES)) ? 1 : 0;
        }))
        return STREAMBP_E_CUDA;
    if (pair) {
        const int pairs = std::max(1, sm_count() / 2);
        const int grid = 2 * (tiles < pairs ? (int)tiles : pairs);
        SBP_LAUNCH(gemm_pair_kernel, grid, NUM_THREADS, PAIR_SMEM_BYTES, st, p);
        return STREAMBP_OK;
    }
    const int grid = tiles < sm_count() ? (int)tiles : sm_count();
    SBP_LAUNCH(gemm_group_kernel, grid, NUM_THREADS, SMEM_BYTES, st, p);
    return STREAMBP_OK;
}

int gemm_tc(GemmOp op, int64_t M, int64_t N, int64_t K, const bf16 *A, int64_t lda, const bf16 *B, int64_t ldb,
            void *C, int64_t ldc, bool c_is_f32, const bf16 *bias, bool accumulate, cudaStream_t st) {
    GemmProb g;
    g.op = op; g.M = M; g.N = N; g.nseg = 1;
    g.seg[0] = GemmSeg{A, lda, B, ldb, K};
    g.C = C; g.ldc = ldc; g.c_is_f32 = c_is_f32; g.bias = bias; g.accumulate = accumulate;
    return gemm_tc_group(&g, 1, nullptr, st);
}

int gemm_tc_take_fault() { return take_fault_local(); }

int gemm_tc_variant() { return !tensor_maps_available() ? 0 : (pair_kernel_available() ? 2 : 1); }

}  // namespace sbp
