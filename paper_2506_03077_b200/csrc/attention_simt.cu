// Partitioned causal GQA attention on CUDA cores (fp32 arithmetic): the queries of one chunk
// against the key/value prefix that ends with the chunk.  Key tiles beyond the diagonal are never
// visited; the mask is applied only inside the tiles the diagonal crosses.  Online softmax with
// warp-shuffle row max / sum; S and P are never stored.  The backward is deterministic: one kernel
// owns a key tile (dK, dV), another owns a query tile (dQ), no floating-point atomics.
//
// Used by the fp32 precision mode and as the reference path for head dims / shapes the tensor-core
// attention does not take.
#include "common.cuh"

namespace sbp {
namespace {

constexpr int BQ = 32, BKV = 32;

template <typename T>
__device__ __forceinline__ void load_tile(float *dst, int ld, const T *src, int64_t row0, int64_t nrows,
                                          int64_t row_stride, int dh) {
    // dst[r][c] = src[(row0 + r) * row_stride + c], r < 32, zero beyond nrows
    const int vec_per_row = dh / 4;
    for (int idx = threadIdx.x; idx < 32 * vec_per_row; idx += blockDim.x) {
        const int r = idx / vec_per_row, c = (idx % vec_per_row) * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (row0 + r < nrows) {
            const T *p = src + (row0 + r) * row_stride + c;
            v = make_float4(to_f32(p[0]), to_f32(p[1]), to_f32(p[2]), to_f32(p[3]));
        }
        *reinterpret_cast<float4 *>(dst + r * ld + c) = v;
    }
}

// s[i] = <Q[w*4+i], K[lane]> for the 4 query rows of warp w
template <int DH>
__device__ __forceinline__ void qk_dots(const float *Qs, const float *Ks, int w, int lane, float s[4]) {
    constexpr int LD = DH + 4;
    s[0] = s[1] = s[2] = s[3] = 0.f;
#pragma unroll 8
    for (int x = 0; x < DH; x += 4) {
        const float4 k4 = *reinterpret_cast<const float4 *>(Ks + lane * LD + x);
#pragma unroll
        for (int i = 0; i < 4; i++) {
            const float4 q4 = *reinterpret_cast<const float4 *>(Qs + (w * 4 + i) * LD + x);
            s[i] += q4.x * k4.x + q4.y * k4.y + q4.z * k4.z + q4.w * k4.w;
        }
    }
}

// ------------------------------------------------------------------------------------------
// forward: grid (query tiles, Hq), 256 threads; warp w owns query rows 4w..4w+3, lane = key column
// ------------------------------------------------------------------------------------------
template <typename T, int DH>
__global__ void __launch_bounds__(256)
    attn_fwd_kernel(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v, int64_t n, int64_t q0,
                    int Hq, int Hkv, T *__restrict__ o, float *__restrict__ lse) {
    pdl_enter();
    constexpr int LD = DH + 4, DPL = DH / 32;  // dims per lane
    extern __shared__ __align__(16) float smem[];
    float *Qs = smem, *Ks = Qs + 32 * LD, *Vs = Ks + 32 * LD;
    const int h = blockIdx.y, g = h / (Hq / Hkv);
    const int64_t qt0 = (int64_t)blockIdx.x * BQ;
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float scale = rsqrtf((float)DH);
    load_tile(Qs, LD, q + (int64_t)h * DH, qt0, n, (int64_t)Hq * DH, DH);
    float m[4], l[4], acc[4][DPL];
#pragma unroll
    for (int i = 0; i < 4; i++) {
        m[i] = -INFINITY;
        l[i] = 0.f;
#pragma unroll
        for (int e = 0; e < DPL; e++) acc[i][e] = 0.f;
    }
    const int64_t last_q_abs = q0 + min(n, qt0 + BQ) - 1;   // last query row of this tile (absolute)
    const int64_t kv_end = last_q_abs + 1;                  // keys 0 .. last_q_abs
    for (int64_t k0 = 0; k0 < kv_end; k0 += BKV) {
        __syncthreads();
        load_tile(Ks, LD, k + (int64_t)g * DH, k0, kv_end, (int64_t)Hkv * DH, DH);
        load_tile(Vs, LD, v + (int64_t)g * DH, k0, kv_end, (int64_t)Hkv * DH, DH);
        __syncthreads();
        float s[4];
        qk_dots<DH>(Qs, Ks, w, lane, s);
        const int64_t kabs = k0 + lane;
#pragma unroll
        for (int i = 0; i < 4; i++) {
            const int64_t qabs = q0 + qt0 + w * 4 + i;
            const bool ok = kabs <= qabs && kabs < kv_end;
            const float sv = ok ? s[i] * scale : -INFINITY;
            const float mt = warp_max(sv);
            const float mn = fmaxf(m[i], mt);          // finite: key 0 is visible to every row
            const float p = ok ? __expf(sv - mn) : 0.f;
            const float corr = __expf(m[i] - mn);
            l[i] = l[i] * corr + warp_sum(p);
            m[i] = mn;
#pragma unroll
            for (int e = 0; e < DPL; e++) acc[i][e] *= corr;
            for (int j = 0; j < BKV; j++) {
                const float pj = __shfl_sync(0xffffffffu, p, j);
#pragma unroll
                for (int e = 0; e < DPL; e++) acc[i][e] += pj * Vs[j * LD + e * 32 + lane];
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 4; i++) {
        const int64_t qr = qt0 + w * 4 + i;
        if (qr >= n) continue;
        const float inv = 1.f / l[i];
#pragma unroll
        for (int e = 0; e < DPL; e++) o[(qr * Hq + h) * DH + e * 32 + lane] = from_f32<T>(acc[i][e] * inv);
        if (lane == 0) lse[(int64_t)h * n + qr] = m[i] + logf(l[i]);
    }
}

// delta[h, i] = sum_j do[i,h,j] * o[i,h,j]; one warp per (i, h)
template <typename T>
__global__ void __launch_bounds__(256)
    attn_delta_kernel(const T *__restrict__ o, const T *__restrict__ dout, int64_t n, int Hq, int dh,
                      float *__restrict__ delta) {
    pdl_enter();
    const int64_t wid = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (wid >= n * Hq) return;
    const int64_t i = wid / Hq;
    const int h = (int)(wid % Hq);
    float acc = 0.f;
    for (int j = lane; j < dh; j += 32) acc += to_f32(o[wid * dh + j]) * to_f32(dout[wid * dh + j]);
    acc = warp_sum(acc);
    if (lane == 0) delta[(int64_t)h * n + i] = acc;
}

// p and ds for the 4 rows of warp w against key `lane` of the tile
template <int DH>
__device__ __forceinline__ void p_and_ds(const float *Qs, const float *dOs, const float *Ks, const float *Vs,
                                         const float *lse_s, const float *delta_s, int w, int lane, int64_t q_abs0,
                                         int64_t n_abs_end, int64_t kabs, int64_t kv_len, float scale, float p[4],
                                         float ds[4]) {
    float s[4], dp[4];
    qk_dots<DH>(Qs, Ks, w, lane, s);
    qk_dots<DH>(dOs, Vs, w, lane, dp);
#pragma unroll
    for (int i = 0; i < 4; i++) {
        const int64_t qabs = q_abs0 + w * 4 + i;
        const bool ok = kabs <= qabs && kabs < kv_len && qabs < n_abs_end;
        p[i] = ok ? __expf(s[i] * scale - lse_s[w * 4 + i]) : 0.f;
        ds[i] = p[i] * (dp[i] - delta_s[w * 4 + i]) * scale;
    }
}

// ------------------------------------------------------------------------------------------
// backward dK/dV: grid (key tiles, Hkv). Thread (kr = tid/8, seg = tid%8) accumulates key row kr,
// dims {seg*4 + 32*e .. +3}.
// ------------------------------------------------------------------------------------------
template <typename T, int DH>
__global__ void __launch_bounds__(256)
    attn_bwd_dkdv_kernel(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v,
                         const T *__restrict__ dout, const float *__restrict__ lse, const float *__restrict__ delta,
                         int64_t n, int64_t q0, int Hq, int Hkv, float *__restrict__ dk, float *__restrict__ dv) {
    pdl_enter();
    constexpr int LD = DH + 4, NE = DH / 32;
    extern __shared__ __align__(16) float smem[];
    float *Ks = smem, *Vs = Ks + 32 * LD, *Qs = Vs + 32 * LD, *dOs = Qs + 32 * LD;
    float *Ps = dOs + 32 * LD, *dSs = Ps + 32 * 33, *lse_s = dSs + 32 * 33, *delta_s = lse_s + 32;
    const int g = blockIdx.y, G = Hq / Hkv;
    const int64_t k0 = (int64_t)blockIdx.x * BKV;
    const int64_t kv_len = q0 + n;
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kr = threadIdx.x >> 3, seg = threadIdx.x & 7;
    const float scale = rsqrtf((float)DH);
    load_tile(Ks, LD, k + (int64_t)g * DH, k0, kv_len, (int64_t)Hkv * DH, DH);
    load_tile(Vs, LD, v + (int64_t)g * DH, k0, kv_len, (int64_t)Hkv * DH, DH);
    float adk[NE][4], adv[NE][4];
#pragma unroll
    for (int e = 0; e < NE; e++)
#pragma unroll
        for (int c = 0; c < 4; c++) adk[e][c] = adv[e][c] = 0.f;
    // first query tile whose last row can see key k0: rows with q0 + r >= k0
    int64_t first_tile = (k0 > q0) ? (k0 - q0) / BQ : 0;
    for (int hh = 0; hh < G; hh++) {
        const int h = g * G + hh;
        for (int64_t qt0 = first_tile * BQ; qt0 < n; qt0 += BQ) {
            __syncthreads();
            load_tile(Qs, LD, q + (int64_t)h * DH, qt0, n, (int64_t)Hq * DH, DH);
            load_tile(dOs, LD, dout + (int64_t)h * DH, qt0, n, (int64_t)Hq * DH, DH);
            if (threadIdx.x < 32) {
                const int64_t r = qt0 + threadIdx.x;
                lse_s[threadIdx.x] = r < n ? lse[(int64_t)h * n + r] : 0.f;
                delta_s[threadIdx.x] = r < n ? delta[(int64_t)h * n + r] : 0.f;
            }
            __syncthreads();
            float p[4], ds[4];
            p_and_ds<DH>(Qs, dOs, Ks, Vs, lse_s, delta_s, w, lane, q0 + qt0, q0 + n, k0 + lane, kv_len, scale, p, ds);
#pragma unroll
            for (int i = 0; i < 4; i++) {
                Ps[(w * 4 + i) * 33 + lane] = p[i];
                dSs[(w * 4 + i) * 33 + lane] = ds[i];
            }
            __syncthreads();
            for (int r = 0; r < BQ; r++) {
                const float pv = Ps[r * 33 + kr], dsv = dSs[r * 33 + kr];
#pragma unroll
                for (int e = 0; e < NE; e++) {
                    const float4 d4 = *reinterpret_cast<const float4 *>(dOs + r * LD + e * 32 + seg * 4);
                    const float4 q4 = *reinterpret_cast<const float4 *>(Qs + r * LD + e * 32 + seg * 4);
                    adv[e][0] += pv * d4.x; adv[e][1] += pv * d4.y; adv[e][2] += pv * d4.z; adv[e][3] += pv * d4.w;
                    adk[e][0] += dsv * q4.x; adk[e][1] += dsv * q4.y; adk[e][2] += dsv * q4.z; adk[e][3] += dsv * q4.w;
                }
            }
        }
    }
    if (k0 + kr < kv_len) {
        float *pk = dk + ((k0 + kr) * Hkv + g) * DH, *pv = dv + ((k0 + kr) * Hkv + g) * DH;
#pragma unroll
        for (int e = 0; e < NE; e++) {
            float4 a = *reinterpret_cast<float4 *>(pk + e * 32 + seg * 4);
            a.x += adk[e][0]; a.y += adk[e][1]; a.z += adk[e][2]; a.w += adk[e][3];
            *reinterpret_cast<float4 *>(pk + e * 32 + seg * 4) = a;
            float4 b = *reinterpret_cast<float4 *>(pv + e * 32 + seg * 4);
            b.x += adv[e][0]; b.y += adv[e][1]; b.z += adv[e][2]; b.w += adv[e][3];
            *reinterpret_cast<float4 *>(pv + e * 32 + seg * 4) = b;
        }
    }
}

// ------------------------------------------------------------------------------------------
// backward dQ: grid (query tiles, Hq). Thread (qr = tid/8, seg = tid%8).
// ------------------------------------------------------------------------------------------
template <typename T, int DH>
__global__ void __launch_bounds__(256)
    attn_bwd_dq_kernel(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v,
                       const T *__restrict__ dout, const float *__restrict__ lse, const float *__restrict__ delta,
                       int64_t n, int64_t q0, int Hq, int Hkv, float *__restrict__ dq) {
    pdl_enter();
    constexpr int LD = DH + 4, NE = DH / 32;
    extern __shared__ __align__(16) float smem[];
    float *Ks = smem, *Vs = Ks + 32 * LD, *Qs = Vs + 32 * LD, *dOs = Qs + 32 * LD;
    float *dSs = dOs + 32 * LD, *lse_s = dSs + 32 * 33, *delta_s = lse_s + 32;
    const int h = blockIdx.y, g = h / (Hq / Hkv);
    const int64_t qt0 = (int64_t)blockIdx.x * BQ;
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int qr = threadIdx.x >> 3, seg = threadIdx.x & 7;
    const float scale = rsqrtf((float)DH);
    load_tile(Qs, LD, q + (int64_t)h * DH, qt0, n, (int64_t)Hq * DH, DH);
    load_tile(dOs, LD, dout + (int64_t)h * DH, qt0, n, (int64_t)Hq * DH, DH);
    if (threadIdx.x < 32) {
        const int64_t r = qt0 + threadIdx.x;
        lse_s[threadIdx.x] = r < n ? lse[(int64_t)h * n + r] : 0.f;
        delta_s[threadIdx.x] = r < n ? delta[(int64_t)h * n + r] : 0.f;
    }
    float adq[NE][4];
#pragma unroll
    for (int e = 0; e < NE; e++)
#pragma unroll
        for (int c = 0; c < 4; c++) adq[e][c] = 0.f;
    const int64_t kv_end = q0 + min(n, qt0 + BQ);
    for (int64_t k0 = 0; k0 < kv_end; k0 += BKV) {
        __syncthreads();
        load_tile(Ks, LD, k + (int64_t)g * DH, k0, kv_end, (int64_t)Hkv * DH, DH);
        load_tile(Vs, LD, v + (int64_t)g * DH, k0, kv_end, (int64_t)Hkv * DH, DH);
        __syncthreads();
        float p[4], ds[4];
        p_and_ds<DH>(Qs, dOs, Ks, Vs, lse_s, delta_s, w, lane, q0 + qt0, q0 + n, k0 + lane, kv_end, scale, p, ds);
#pragma unroll
        for (int i = 0; i < 4; i++) dSs[(w * 4 + i) * 33 + lane] = ds[i];
        __syncthreads();
        for (int j = 0; j < BKV; j++) {
            const float dsv = dSs[qr * 33 + j];
#pragma unroll
            for (int e = 0; e < NE; e++) {
                const float4 k4 = *reinterpret_cast<const float4 *>(Ks + j * LD + e * 32 + seg * 4);
                adq[e][0] += dsv * k4.x; adq[e][1] += dsv * k4.y; adq[e][2] += dsv * k4.z; adq[e][3] += dsv * k4.w;
            }
        }
    }
    if (qt0 + qr < n) {
        float *pq = dq + ((qt0 + qr) * Hq + h) * DH;
#pragma unroll
        for (int e = 0; e < NE; e++)
            *reinterpret_cast<float4 *>(pq + e * 32 + seg * 4) = make_float4(adq[e][0], adq[e][1], adq[e][2], adq[e][3]);
    }
}

template <typename K>
bool set_smem(K kernel, size_t bytes) {
    return cuda_ok(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
}

}  // namespace

template <typename T>
int attention_fwd(const T *q, const T *k, const T *v, int64_t n, int64_t q0, int Hq, int Hkv, int dh, T *o, float *lse,
                  cudaStream_t st) {
    if (n <= 0) return STREAMBP_OK;
    dim3 grid((unsigned)((n + BQ - 1) / BQ), Hq);
    const size_t smem = (size_t)3 * 32 * (dh + 4) * sizeof(float);
    if (dh == 128) {
        if (!set_smem(attn_fwd_kernel<T, 128>, smem)) return STREAMBP_E_CUDA;
        SBP_LAUNCH((attn_fwd_kernel<T, 128>), grid, 256, smem, st, q, k, v, n, q0, Hq, Hkv, o, lse);
    } else if (dh == 64) {
        if (!set_smem(attn_fwd_kernel<T, 64>, smem)) return STREAMBP_E_CUDA;
        SBP_LAUNCH((attn_fwd_kernel<T, 64>), grid, 256, smem, st, q, k, v, n, q0, Hq, Hkv, o, lse);
    } else {
        return STREAMBP_E_SHAPE;
    }
    return STREAMBP_OK;
}

template <typename T>
int attention_bwd(const T *q, const T *k, const T *v, const T *o, const T *dout, const float *lse, int64_t n,
                  int64_t q0, int Hq, int Hkv, int dh, float *delta, float *dq, float *dk, float *dv, cudaStream_t st) {
    if (n <= 0) return STREAMBP_OK;
    const int64_t kv_len = q0 + n;
    {
        const int64_t warps = n * Hq;
        SBP_LAUNCH(attn_delta_kernel<T>, (unsigned)((warps * 32 + 255) / 256), 256, 0, st, o, dout, n, Hq, dh, delta);
    }
    dim3 gkv((unsigned)((kv_len + BKV - 1) / BKV), Hkv);
    dim3 gq((unsigned)((n + BQ - 1) / BQ), Hq);
    const size_t smem = ((size_t)4 * 32 * (dh + 4) + 2 * 32 * 33 + 64) * sizeof(float);
    if (dh == 128) {
        if (!set_smem(attn_bwd_dkdv_kernel<T, 128>, smem) || !set_smem(attn_bwd_dq_kernel<T, 128>, smem))
            return STREAMBP_E_CUDA;
        SBP_LAUNCH((attn_bwd_dkdv_kernel<T, 128>), gkv, 256, smem, st, q, k, v, dout, lse, delta, n, q0, Hq, Hkv, dk, dv);
        SBP_LAUNCH((attn_bwd_dq_kernel<T, 128>), gq, 256, smem, st, q, k, v, dout, lse, delta, n, q0, Hq, Hkv, dq);
    } else if (dh == 64) {
        if (!set_smem(attn_bwd_dkdv_kernel<T, 64>, smem) || !set_smem(attn_bwd_dq_kernel<T, 64>, smem))
            return STREAMBP_E_CUDA;
        SBP_LAUNCH((attn_bwd_dkdv_kernel<T, 64>), gkv, 256, smem, st, q, k, v, dout, lse, delta, n, q0, Hq, Hkv, dk, dv);
        SBP_LAUNCH((attn_bwd_dq_kernel<T, 64>), gq, 256, smem, st, q, k, v, dout, lse, delta, n, q0, Hq, Hkv, dq);
    } else {
        return STREAMBP_E_SHAPE;
    }
    return STREAMBP_OK;
}

template <typename T>
int attention_delta(const T *o, const T *dout, int64_t n, int Hq, int dh, float *delta, cudaStream_t st) {
    if (n <= 0) return STREAMBP_OK;
    const int64_t warps = n * Hq;
    SBP_LAUNCH(attn_delta_kernel<T>, (unsigned)((warps * 32 + 255) / 256), 256, 0, st, o, dout, n, Hq, dh, delta);
    return STREAMBP_OK;
}
template int attention_delta<float>(const float *, const float *, int64_t, int, int, float *, cudaStream_t);
template int attention_delta<bf16>(const bf16 *, const bf16 *, int64_t, int, int, float *, cudaStream_t);

template int attention_fwd<float>(const float *, const float *, const float *, int64_t, int64_t, int, int, int, float *,
                                  float *, cudaStream_t);
template int attention_fwd<bf16>(const bf16 *, const bf16 *, const bf16 *, int64_t, int64_t, int, int, int, bf16 *,
                                 float *, cudaStream_t);
template int attention_bwd<float>(const float *, const float *, const float *, const float *, const float *,
                                  const float *, int64_t, int64_t, int, int, int, float *, float *, float *, float *,
                                  cudaStream_t);
template int attention_bwd<bf16>(const bf16 *, const bf16 *, const bf16 *, const bf16 *, const bf16 *, const float *,
                                 int64_t, int64_t, int, int, int, float *, float *, float *, float *, cudaStream_t);

}  // namespace sbp
