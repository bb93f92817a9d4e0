// fp32-accurate CUDA-core GEMM used by the fp32 precision mode (a single-pass TF32 tensor-core
// product cannot hold 1e-4 relative error) and as the always-available fallback for shapes the
// tcgen05 kernel does not take.  64x64 output tile, 16-deep K slices, 4x4 micro-tile per thread,
// fp32 FMA accumulation.  Three operand layouts (see GemmOp).
#include "common.cuh"

namespace sbp {

namespace {
constexpr int BM = 64, BN = 64, BK = 16, LDS = 68;

// A element (m,k) at A[m*sam + k*sak]; B element (k,n) at B[k*sbk + n*sbn]
template <typename TI, typename TC, bool A_KCONTIG, bool B_KCONTIG>
__global__ void __launch_bounds__(256)
    gemm_simt_kernel(int64_t M, int64_t N, int64_t K, const TI *__restrict__ A, int64_t sam, int64_t sak,
                     const TI *__restrict__ B, int64_t sbk, int64_t sbn, TC *C, int64_t ldc,
                     const TI *__restrict__ bias, int accumulate, const int *gate) {
    pdl_enter();
    __shared__ __align__(16) float As[BK][LDS];
    if (gated_off(gate)) return;
    __shared__ __align__(16) float Bs[BK][LDS];
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int64_t m0 = (int64_t)blockIdx.y * BM, n0 = (int64_t)blockIdx.x * BN;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; i++)
#pragma unroll
        for (int j = 0; j < 4; j++) acc[i][j] = 0.f;

    for (int64_t k0 = 0; k0 < K; k0 += BK) {
#pragma unroll
        for (int e = 0; e < 4; e++) {
            const int idx = tid + e * 256;
            int m, k;
            if (A_KCONTIG) { m = idx >> 4; k = idx & 15; } else { k = idx >> 6; m = idx & 63; }
            const int64_t gm = m0 + m, gk = k0 + k;
            As[k][m] = (gm < M && gk < K) ? to_f32(A[gm * sam + gk * sak]) : 0.f;
            int n, kb;
            if (B_KCONTIG) { n = idx >> 4; kb = idx & 15; } else { kb = idx >> 6; n = idx & 63; }
            const int64_t gn = n0 + n, gkb = k0 + kb;
            Bs[kb][n] = (gn < N && gkb < K) ? to_f32(B[gkb * sbk + gn * sbn]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; k++) {
            const float4 a4 = *reinterpret_cast<const float4 *>(&As[k][ty * 4]);
            const float4 b4 = *reinterpret_cast<const float4 *>(&Bs[k][tx * 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int i = 0; i < 4; i++)
#pragma unroll
                for (int j = 0; j < 4; j++) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; i++) {
        const int64_t gm = m0 + ty * 4 + i;
        if (gm >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; j++) {
            const int64_t gn = n0 + tx * 4 + j;
            if (gn >= N) continue;
            float v = acc[i][j];
            if (bias) v += to_f32(bias[gn]);
            if (accumulate) v += to_f32(C[gm * ldc + gn]);
            C[gm * ldc + gn] = from_f32<TC>(v);
        }
    }
}
}  // namespace

template <typename TI, typename TC>
int gemm(GemmOp op, int64_t M, int64_t N, int64_t K, const TI *A, int64_t lda, const TI *B, int64_t ldb, TC *C,
         int64_t ldc, const TI *bias, bool accumulate, cudaStream_t st) {
    if (M <= 0 || N <= 0) return STREAMBP_OK;
    dim3 grid((unsigned)((N + BN - 1) / BN), (unsigned)((M + BM - 1) / BM));
    const int acc = accumulate ? 1 : 0;
    switch (op) {
        case OP_NT:
            SBP_LAUNCH((gemm_simt_kernel<TI, TC, true, true>), grid, 256, 0, st, M, N, K, A, lda, (int64_t)1, B,
                       (int64_t)1, ldb, C, ldc, bias, acc, call_state().gate);
            break;
        case OP_NN:
            SBP_LAUNCH((gemm_simt_kernel<TI, TC, true, false>), grid, 256, 0, st, M, N, K, A, lda, (int64_t)1, B, ldb,
                       (int64_t)1, C, ldc, bias, acc, call_state().gate);
            break;
        case OP_TN:
            SBP_LAUNCH((gemm_simt_kernel<TI, TC, false, false>), grid, 256, 0, st, M, N, K, A, (int64_t)1, lda, B, ldb,
                       (int64_t)1, C, ldc, bias, acc, call_state().gate);
            break;
    }
    return STREAMBP_OK;
}

template int gemm<float, float>(GemmOp, int64_t, int64_t, int64_t, const float *, int64_t, const float *, int64_t,
                                float *, int64_t, const float *, bool, cudaStream_t);
template int gemm<bf16, float>(GemmOp, int64_t, int64_t, int64_t, const bf16 *, int64_t, const bf16 *, int64_t,
                               float *, int64_t, const bf16 *, bool, cudaStream_t);
template int gemm<bf16, bf16>(GemmOp, int64_t, int64_t, int64_t, const bf16 *, int64_t, const bf16 *, int64_t, bf16 *,
                              int64_t, const bf16 *, bool, cudaStream_t);

}  // namespace sbp
