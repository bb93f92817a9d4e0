// HBM-bound steps of the streamed backward: RMSNorm forward/backward, RoPE, SwiGLU,
// column sums, casts, cross-entropy rows, embedding gather / scatter-add.
// All kernels move 16 bytes per thread per access and reduce rows with warp shuffles.
#include <algorithm>

#include "common.cuh"

namespace sbp {

// ---------------------------------------------------------------------------------
// RMSNorm forward: one block per row.
// ---------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) rmsnorm_fwd_kernel(const T *__restrict__ x, const float *__restrict__ res,
                                                          const T *__restrict__ gain, float eps, int d,
                                                          T *__restrict__ h, float *__restrict__ rstd_out,
                                                          float *__restrict__ r_out, const int *gate) {
    pdl_enter();
    __shared__ float red[33];
    if (gated_off(gate)) return;
    const int64_t row = blockIdx.x;
    const T *xr = x + row * d;
    constexpr int N = Vec<T>::N;
    float ss = 0.f;
    for (int c = threadIdx.x * N; c < d; c += blockDim.x * N) {
        Vec<T> a;
        a.load(xr + c);
        if (res) {
#pragma unroll
            for (int i = 0; i < N; i += 4) {
                float4 r4 = *reinterpret_cast<const float4 *>(res + row * d + c + i);
                a.v[i] += r4.x; a.v[i + 1] += r4.y; a.v[i + 2] += r4.z; a.v[i + 3] += r4.w;
                *reinterpret_cast<float4 *>(r_out + row * d + c + i) =
                    make_float4(a.v[i], a.v[i + 1], a.v[i + 2], a.v[i + 3]);
            }
        }
#pragma unroll
        for (int i = 0; i < N; i++) ss += a.v[i] * a.v[i];
    }
    ss = block_sum(ss, red);
    const float rstd = rsqrtf(ss / (float)d + eps);
    if (threadIdx.x == 0) rstd_out[row] = rstd;
    for (int c = threadIdx.x * N; c < d; c += blockDim.x * N) {
        Vec<T> a, g, o;
        if (res) {
#pragma unroll
            for (int i = 0; i < N; i += 4) {
                float4 r4 = *reinterpret_cast<const float4 *>(r_out + row * d + c + i);
                a.v[i] = r4.x; a.v[i + 1] = r4.y; a.v[i + 2] = r4.z; a.v[i + 3] = r4.w;
            }
        } else {
            a.load(xr + c);
        }
        g.load(gain + c);
#pragma unroll
        for (int i = 0; i < N; i++) o.v[i] = a.v[i] * rstd * g.v[i];
        o.store(h + row * d + c);
    }
}

template <typename T>
int rmsnorm_fwd(const T *x, const float *res, const T *gain, float eps, int64_t rows, int d, T *h, float *rstd,
                float *r_out, cudaStream_t st) {
    if (rows <= 0) return STREAMBP_OK;
    SBP_LAUNCH(rmsnorm_fwd_kernel<T>, (unsigned)rows, 256, 0, st, x, res, gain, eps, d, h, rstd, r_out,
               call_state().gate);
    return STREAMBP_OK;
}
template int rmsnorm_fwd<float>(const float *, const float *, const float *, float, int64_t, int, float *, float *,
                                float *, cudaStream_t);
template int rmsnorm_fwd<bf16>(const bf16 *, const float *, const bf16 *, float, int64_t, int, bf16 *, float *,
                               float *, cudaStream_t);

// four consecutive values of a row in one store (the row base and the column are multiples of 4 elements)
__device__ __forceinline__ void store4(float *p, const float (&o)[4]) {
    *reinterpret_cast<float4 *>(p) = make_float4(o[0], o[1], o[2], o[3]);
}
__device__ __forceinline__ void store4(bf16 *p, const float (&o)[4]) {
    __nv_bfloat162 a = __floats2bfloat162_rn(o[0], o[1]), b = __floats2bfloat162_rn(o[2], o[3]);
    *reinterpret_cast<uint2 *>(p) = make_uint2(*reinterpret_cast<uint32_t *>(&a), *reinterpret_cast<uint32_t *>(&b));
}

__device__ __forceinline__ void load4(const float *p, float (&o)[4]) {
    const float4 t = *reinterpret_cast<const float4 *>(p);
    o[0] = t.x; o[1] = t.y; o[2] = t.z; o[3] = t.w;
}
__device__ __forceinline__ void load4(const bf16 *p, float (&o)[4]) {
    const uint2 t = *reinterpret_cast<const uint2 *>(p);
    o[0] = __uint_as_float(t.x << 16); o[1] = __uint_as_float(t.x & 0xFFFF0000u);
    o[2] = __uint_as_float(t.y << 16); o[3] = __uint_as_float(t.y & 0xFFFF0000u);
}

// ---------------------------------------------------------------------------------
// RMSNorm backward, row part: out = add + ((dh*g) - xhat * mean((dh*g)*xhat)) * rstd
// ---------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
    rmsnorm_bwd_rows_kernel(const float *__restrict__ dh, const T *__restrict__ xT, const float *__restrict__ xF,
                            const float *__restrict__ rstd_in, const T *__restrict__ gain,
                            const T *__restrict__ addT, const float *__restrict__ addF, int d,
                            float *__restrict__ outF, T *__restrict__ outT, const int *gate) {
    pdl_enter();
    __shared__ float red[33];
    const int64_t row = blockIdx.x;
    if (gated_off(gate)) {   // the upstream gradient of this block of rows is exactly zero
        for (int c = threadIdx.x; c < d; c += blockDim.x) {
            if (outF) outF[row * d + c] = 0.f;
            if (outT) outT[row * d + c] = from_f32<T>(0.f);
        }
        return;
    }
    const float rstd = rstd_in[row];
    float dot = 0.f;
    for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {     // d is a multiple of 4 (of 8 at the C ABI)
        float gh[4], xv[4], gn[4];
        load4(dh + row * d + c, gh);
        if (xF) load4(xF + row * d + c, xv);
        else load4(xT + row * d + c, xv);
        load4(gain + c, gn);
#pragma unroll
        for (int i = 0; i < 4; i++) dot += gh[i] * gn[i] * xv[i] * rstd;
    }
    dot = block_sum(dot, red);
    const float mean = dot / (float)d;
    for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {
        float gh[4], xv[4], gn[4], o[4];
        load4(dh + row * d + c, gh);
        if (xF) load4(xF + row * d + c, xv);
        else load4(xT + row * d + c, xv);
        load4(gain + c, gn);
#pragma unroll
        for (int i = 0; i < 4; i++) o[i] = (gh[i] * gn[i] - xv[i] * rstd * mean) * rstd;
        if (addF) {
            float t[4];
            load4(addF + row * d + c, t);
#pragma unroll
            for (int i = 0; i < 4; i++) o[i] += t[i];
        }
        if (addT) {
            float t[4];
            load4(addT + row * d + c, t);
#pragma unroll
            for (int i = 0; i < 4; i++) o[i] += t[i];
        }
        if (outF) store4(outF + row * d + c, o);
        if (outT) store4(outT + row * d + c, o);
    }
}

// dgain partials: block (col block of 256, row split); partial[split, col] = sum_t dh*x*rstd
template <typename T>
__global__ void __launch_bounds__(256)
    rmsnorm_dgain_partial_kernel(const float *__restrict__ dh, const T *__restrict__ xT, const float *__restrict__ xF,
                                 const float *__restrict__ rstd, int64_t rows, int d, int rows_per_split,
                                 float *__restrict__ partial, const int *gate) {
    pdl_enter();
    const int col = blockIdx.x * 256 + threadIdx.x;
    if (col >= d || gated_off(gate)) return;
    const int64_t r0 = (int64_t)blockIdx.y * rows_per_split;
    const int64_t r1 = min(rows, r0 + (int64_t)rows_per_split);
    float acc = 0.f;
    for (int64_t r = r0; r < r1; r++) {
        const float xv = xF ? xF[r * d + col] : to_f32(xT[r * d + col]);
        acc += dh[r * d + col] * xv * rstd[r];
    }
    partial[(int64_t)blockIdx.y * d + col] = acc;
}

__global__ void __launch_bounds__(256)
    partial_reduce_kernel(const float *__restrict__ partial, int nsplit, int cols, float *__restrict__ out,
                          int accumulate, const int *gate) {
    pdl_enter();
    const int col = blockIdx.x * 256 + threadIdx.x;
    if (col >= cols || gated_off(gate)) return;
    float acc = 0.f;
    for (int s = 0; s < nsplit; s++) acc += partial[(int64_t)s * cols + col];
    out[col] = accumulate ? out[col] + acc : acc;
}

static inline int split_count(int64_t rows) {
    int64_t n = (rows + 31) / 32;
    return (int)(n < 1 ? 1 : (n > 64 ? 64 : n));
}
int rmsnorm_bwd_partials_rows(int64_t rows) { return split_count(rows); }
int colsum_partial_rows(int64_t rows) { return split_count(rows); }

template <typename T>
int rmsnorm_bwd(const float *dh, const T *xT, const float *xF, const float *rstd, const T *gain, const T *addT,
                const float *addF, int64_t rows, int d, float *outF, T *outT, float *dgain, float *partials,
                cudaStream_t st) {
    if (rows <= 0) return STREAMBP_OK;
    const int *gate = call_state().gate;
    SBP_LAUNCH(rmsnorm_bwd_rows_kernel<T>, (unsigned)rows, 256, 0, st, dh, xT, xF, rstd, gain, addT, addF, d, outF,
               outT, gate);
    if (dgain) {
        const int ns = split_count(rows);
        const int rps = (int)((rows + ns - 1) / ns);
        dim3 grid((d + 255) / 256, ns);
        SBP_LAUNCH(rmsnorm_dgain_partial_kernel<T>, grid, 256, 0, st, dh, xT, xF, rstd, rows, d, rps, partials, gate);
        SBP_LAUNCH(partial_reduce_kernel, (d + 255) / 256, 256, 0, st, partials, ns, d, dgain, 1, gate);
    }
    return STREAMBP_OK;
}
template int rmsnorm_bwd<float>(const float *, const float *, const float *, const float *, const float *,
                                const float *, const float *, int64_t, int, float *, float *, float *, float *,
                                cudaStream_t);
template int rmsnorm_bwd<bf16>(const float *, const bf16 *, const float *, const float *, const bf16 *, const bf16 *,
                               const float *, int64_t, int, float *, bf16 *, float *, float *, cudaStream_t);

// ---------------------------------------------------------------------------------
// column sums (bias gradients)
// ---------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
    colsum_partial_kernel(const T *__restrict__ a, int64_t rows, int cols, int rows_per_split,
                          float *__restrict__ partial) {
    pdl_enter();
    const int col = blockIdx.x * 256 + threadIdx.x;
    if (col >= cols) return;
    const int64_t r0 = (int64_t)blockIdx.y * rows_per_split;
    const int64_t r1 = min(rows, r0 + (int64_t)rows_per_split);
    float acc = 0.f;
    for (int64_t r = r0; r < r1; r++) acc += to_f32(a[r * cols + col]);
    partial[(int64_t)blockIdx.y * cols + col] = acc;
}

template <typename T>
int colsum(const T *a, int64_t rows, int cols, float *out, bool accumulate, float *partials, cudaStream_t st) {
    if (rows <= 0) return STREAMBP_OK;
    const int ns = split_count(rows);
    const int rps = (int)((rows + ns - 1) / ns);
    dim3 grid((cols + 255) / 256, ns);
    SBP_LAUNCH(colsum_partial_kernel<T>, grid, 256, 0, st, a, rows, cols, rps, partials);
    SBP_LAUNCH(partial_reduce_kernel, (cols + 255) / 256, 256, 0, st, partials, ns, cols, out, accumulate ? 1 : 0,
               (const int *)nullptr);
    return STREAMBP_OK;
}
// The three bias gradients of a chunk (column sums of dq, dk, dv) in one pair of launches: the column index runs
// over the concatenation of the three matrices.
template <typename T>
struct Colsum3 {
    const T *a[3];
    float *out[3];
    int cols[3];
};
template <typename T>
__global__ void __launch_bounds__(256)
    colsum3_partial_kernel(const Colsum3<T> q, int64_t rows, int rows_per_split, float *__restrict__ partial) {
    pdl_enter();
    const int total = q.cols[0] + q.cols[1] + q.cols[2];
    int col = blockIdx.x * 256 + threadIdx.x;
    if (col >= total) return;
    const int gcol = col;
    int m = 0;
    if (col >= q.cols[0]) { col -= q.cols[0]; m = 1; }
    if (m == 1 && col >= q.cols[1]) { col -= q.cols[1]; m = 2; }
    const T *a = m == 0 ? q.a[0] : (m == 1 ? q.a[1] : q.a[2]);
    const int cols = m == 0 ? q.cols[0] : (m == 1 ? q.cols[1] : q.cols[2]);
    const int64_t r0 = (int64_t)blockIdx.y * rows_per_split;
    const int64_t r1 = min(rows, r0 + (int64_t)rows_per_split);
    float acc = 0.f;
    for (int64_t r = r0; r < r1; r++) acc += to_f32(a[r * cols + col]);
    partial[(int64_t)blockIdx.y * total + gcol] = acc;
}
template <typename T>
__global__ void __launch_bounds__(256)
    colsum3_reduce_kernel(const Colsum3<T> q, const float *__restrict__ partial, int nsplit) {
    pdl_enter();
    const int total = q.cols[0] + q.cols[1] + q.cols[2];
    int col = blockIdx.x * 256 + threadIdx.x;
    if (col >= total) return;
    float acc = 0.f;
    for (int s = 0; s < nsplit; s++) acc += partial[(int64_t)s * total + col];
    int m = 0;
    if (col >= q.cols[0]) { col -= q.cols[0]; m = 1; }
    if (m == 1 && col >= q.cols[1]) { col -= q.cols[1]; m = 2; }
    float *out = m == 0 ? q.out[0] : (m == 1 ? q.out[1] : q.out[2]);
    out[col] += acc;
}
template <typename T>
int colsum3_add(const T *a0, int c0, float *o0, const T *a1, int c1, float *o1, const T *a2, int c2, float *o2,
                int64_t rows, float *partials, cudaStream_t st) {
    if (rows <= 0) return STREAMBP_OK;
    Colsum3<T> q{{a0, a1, a2}, {o0, o1, o2}, {c0, c1, c2}};
    const int total = c0 + c1 + c2;
    const int ns = split_count(rows);
    const int rps = (int)((rows + ns - 1) / ns);
    dim3 grid((total + 255) / 256, ns);
    SBP_LAUNCH(colsum3_partial_kernel<T>, grid, 256, 0, st, q, rows, rps, partials);
    SBP_LAUNCH(colsum3_reduce_kernel<T>, (total + 255) / 256, 256, 0, st, q, partials, ns);
    return STREAMBP_OK;
}
template int colsum3_add<float>(const float *, int, float *, const float *, int, float *, const float *, int, float *,
                                int64_t, float *, cudaStream_t);
template int colsum3_add<bf16>(const bf16 *, int, float *, const bf16 *, int, float *, const bf16 *, int, float *,
                               int64_t, float *, cudaStream_t);

template int colsum<float>(const float *, int64_t, int, float *, bool, float *, cudaStream_t);
template int colsum<bf16>(const bf16 *, int64_t, int, float *, bool, float *, cudaStream_t);

// ---------------------------------------------------------------------------------
// RoPE: table of (cos, sin) built in double precision, applied in fp32.
// ---------------------------------------------------------------------------------
__global__ void rope_table_kernel(float2 *__restrict__ cs, int64_t pos0, int64_t rows, int half, double theta) {
    pdl_enter();
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * half) return;
    const int64_t t = idx / half;
    const int j = (int)(idx % half);
    const double inv_freq = pow(theta, -(double)j / (double)half);
    double s, c;
    sincos((double)(pos0 + t) * inv_freq, &s, &c);
    cs[idx] = make_float2((float)c, (float)s);
}

int rope_table(float *cs, int64_t pos0, int64_t rows, int dh, float theta, cudaStream_t st) {
    const int half = dh / 2;
    const int64_t n = rows * half;
    if (n <= 0) return STREAMBP_OK;
    SBP_LAUNCH(rope_table_kernel, (unsigned)((n + 255) / 256), 256, 0, st, reinterpret_cast<float2 *>(cs), pos0, rows,
               half, (double)theta);
    return STREAMBP_OK;
}

// thread = 4 consecutive frequencies j of one (row, head): reads 2 x float4, writes 2 x 4 values
template <typename TO>
__global__ void __launch_bounds__(256)
    rope_apply_kernel(const float *__restrict__ in, const float2 *__restrict__ cs, int64_t rows, int heads, int dh,
                      int transpose, TO *__restrict__ out) {
    pdl_enter();
    const int half = dh / 2, q4 = half / 4;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * heads * q4) return;
    const int j = (int)(idx % q4) * 4;
    const int64_t th = idx / q4;
    const int64_t t = th / heads;
    const float *p = in + th * dh;
    const float4 a = *reinterpret_cast<const float4 *>(p + j);
    const float4 b = *reinterpret_cast<const float4 *>(p + half + j);
    const float4 cs0 = *reinterpret_cast<const float4 *>(cs + t * half + j);
    const float4 cs1 = *reinterpret_cast<const float4 *>(cs + t * half + j + 2);
    const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
    const float c[4] = {cs0.x, cs0.z, cs1.x, cs1.z};
    float s[4] = {cs0.y, cs0.w, cs1.y, cs1.w};
    if (transpose) {
#pragma unroll
        for (int i = 0; i < 4; i++) s[i] = -s[i];
    }
    TO *o = out + th * dh;
#pragma unroll
    for (int i = 0; i < 4; i++) {
        o[j + i] = from_f32<TO>(av[i] * c[i] - bv[i] * s[i]);
        o[half + j + i] = from_f32<TO>(bv[i] * c[i] + av[i] * s[i]);
    }
}

template <typename TO>
int rope_apply(const float *in, const float *cs, int64_t rows, int heads, int dh, bool transpose, TO *out,
               cudaStream_t st) {
    const int64_t n = rows * heads * (dh / 8);
    if (n <= 0) return STREAMBP_OK;
    SBP_LAUNCH(rope_apply_kernel<TO>, (unsigned)((n + 255) / 256), 256, 0, st, in, reinterpret_cast<const float2 *>(cs),
               rows, heads, dh, transpose ? 1 : 0, out);
    return STREAMBP_OK;
}
template int rope_apply<float>(const float *, const float *, int64_t, int, int, bool, float *, cudaStream_t);
template int rope_apply<bf16>(const float *, const float *, int64_t, int, int, bool, bf16 *, cudaStream_t);

// ---------------------------------------------------------------------------------
// SwiGLU
// ---------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) swiglu_fwd_kernel(const T *__restrict__ g, const T *__restrict__ u, int64_t n,
                                                         T *__restrict__ m) {
    pdl_enter();
    constexpr int N = Vec<T>::N;
    const int64_t i0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * N;
    if (i0 >= n) return;
    Vec<T> a, b, o;
    a.load(g + i0);
    b.load(u + i0);
#pragma unroll
    for (int i = 0; i < N; i++) {
        const float sg = 1.f / (1.f + __expf(-a.v[i]));
        o.v[i] = a.v[i] * sg * b.v[i];
    }
    o.store(m + i0);
}
template <typename T>
__global__ void __launch_bounds__(256) swiglu_bwd_kernel(const T *__restrict__ dm, T *__restrict__ g, T *__restrict__ u,
                                                         int64_t n) {
    pdl_enter();
    constexpr int N = Vec<T>::N;
    const int64_t i0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * N;
    if (i0 >= n) return;
    Vec<T> a, b, c, og, ou;
    a.load(g + i0);
    b.load(u + i0);
    c.load(dm + i0);
#pragma unroll
    for (int i = 0; i < N; i++) {
        const float sg = 1.f / (1.f + __expf(-a.v[i]));
        ou.v[i] = c.v[i] * a.v[i] * sg;                                      // du = dm * silu(g)
        og.v[i] = c.v[i] * b.v[i] * sg * (1.f + a.v[i] * (1.f - sg));        // dg = dm * u * silu'(g)
    }
    og.store(g + i0);
    ou.store(u + i0);
}
template <typename T>
int swiglu_fwd(const T *g, const T *u, int64_t n, T *m, cudaStream_t st) {
    if (n <= 0) return STREAMBP_OK;
    const int64_t nv = n / Vec<T>::N;
    SBP_LAUNCH(swiglu_fwd_kernel<T>, (unsigned)((nv + 255) / 256), 256, 0, st, g, u, n, m);
    return STREAMBP_OK;
}
template <typename T>
int swiglu_bwd(const T *dm, T *g, T *u, int64_t n, cudaStream_t st) {
    if (n <= 0) return STREAMBP_OK;
    const int64_t nv = n / Vec<T>::N;
    SBP_LAUNCH(swiglu_bwd_kernel<T>, (unsigned)((nv + 255) / 256), 256, 0, st, dm, g, u, n);
    return STREAMBP_OK;
}
template int swiglu_fwd<float>(const float *, const float *, int64_t, float *, cudaStream_t);
template int swiglu_fwd<bf16>(const bf16 *, const bf16 *, int64_t, bf16 *, cudaStream_t);
template int swiglu_bwd<float>(const float *, float *, float *, int64_t, cudaStream_t);
template int swiglu_bwd<bf16>(const bf16 *, bf16 *, bf16 *, int64_t, cudaStream_t);

// ---------------------------------------------------------------------------------
// casts / fills
// ---------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) cast_kernel(const float *__restrict__ in, int64_t n, T *__restrict__ out) {
    pdl_enter();
    const int64_t i0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i0 >= n) return;
    const float4 a = *reinterpret_cast<const float4 *>(in + i0);
    out[i0] = from_f32<T>(a.x);
    out[i0 + 1] = from_f32<T>(a.y);
    out[i0 + 2] = from_f32<T>(a.z);
    out[i0 + 3] = from_f32<T>(a.w);
}
template <typename T>
int cast_from_f32(const float *in, int64_t n, T *out, cudaStream_t st) {
    if (n <= 0) return STREAMBP_OK;
    SBP_LAUNCH(cast_kernel<T>, (unsigned)((n / 4 + 255) / 256), 256, 0, st, in, n, out);
    return STREAMBP_OK;
}
template int cast_from_f32<float>(const float *, int64_t, float *, cudaStream_t);
template int cast_from_f32<bf16>(const float *, int64_t, bf16 *, cudaStream_t);

template <typename T>
__global__ void __launch_bounds__(256) add_cast_kernel(const float *__restrict__ a, const float *__restrict__ b,
                                                       int64_t n, T *__restrict__ out) {
    pdl_enter();
    const int64_t i0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i0 >= n) return;
    const float4 x = *reinterpret_cast<const float4 *>(a + i0);
    const float4 y = *reinterpret_cast<const float4 *>(b + i0);
    out[i0] = from_f32<T>(x.x + y.x);
    out[i0 + 1] = from_f32<T>(x.y + y.y);
    out[i0 + 2] = from_f32<T>(x.z + y.z);
    out[i0 + 3] = from_f32<T>(x.w + y.w);
}
template <typename T>
int add_cast(const float *a, const float *b, int64_t n, T *out, cudaStream_t st) {
    if (n <= 0) return STREAMBP_OK;
    SBP_LAUNCH(add_cast_kernel<T>, (unsigned)((n / 4 + 255) / 256), 256, 0, st, a, b, n, out);
    return STREAMBP_OK;
}
template int add_cast<float>(const float *, const float *, int64_t, float *, cudaStream_t);
template int add_cast<bf16>(const float *, const float *, int64_t, bf16 *, cudaStream_t);

// ---- workspace guards (debug mode) ---------------------------------------------------------------
namespace {
constexpr int kGuardsPerLaunch = 48;
struct GuardList {
    unsigned long long off[kGuardsPerLaunch];
    int first, n;
};
__device__ __forceinline__ uint32_t guard_word(int guard, int word) { return 0xA5C3F00Du ^ ((uint32_t)guard * 2654435761u) ^ (uint32_t)word; }
__global__ void guards_arm_kernel(char *base, GuardList g) {
    pdl_enter();
    uint32_t *p = reinterpret_cast<uint32_t *>(base + g.off[blockIdx.x]);
    p[threadIdx.x] = guard_word(g.first + blockIdx.x, threadIdx.x);
}
__global__ void guards_check_kernel(const char *base, GuardList g, WsHeader *hdr) {
    pdl_enter();
    const uint32_t *p = reinterpret_cast<const uint32_t *>(base + g.off[blockIdx.x]);
    if (p[threadIdx.x] != guard_word(g.first + blockIdx.x, threadIdx.x)) set_status(hdr, STREAMBP_E_WORKSPACE_GUARD, g.first + blockIdx.x);
}
template <typename F>
int for_guard_batches(const std::vector<size_t> &guards, F launch) {
    for (size_t i = 0; i < guards.size(); i += kGuardsPerLaunch) {
        GuardList g;
        g.first = (int)i;
        g.n = (int)std::min<size_t>(kGuardsPerLaunch, guards.size() - i);
        for (int k = 0; k < g.n; k++) g.off[k] = guards[i + k];
        SBP_TRY(launch(g));
    }
    return STREAMBP_OK;
}
}  // namespace

int ws_guards_arm(void *base, const std::vector<size_t> &guards, cudaStream_t st) {
    return for_guard_batches(guards, [&](const GuardList &g) -> int {
        SBP_LAUNCH(guards_arm_kernel, g.n, (int)(kGuardBytes / 4), 0, st, static_cast<char *>(base), g);
        return (int)STREAMBP_OK;
    });
}
int ws_guards_check(void *base, const std::vector<size_t> &guards, WsHeader *hdr, cudaStream_t st) {
    return for_guard_batches(guards, [&](const GuardList &g) -> int {
        SBP_LAUNCH(guards_check_kernel, g.n, (int)(kGuardBytes / 4), 0, st, static_cast<const char *>(base), g, hdr);
        return (int)STREAMBP_OK;
    });
}

// test hook: `overrun` floats written past the end of a buffer of `count` floats
__global__ void overrun_kernel(float *buf, int count, int overrun) {
    pdl_enter();
    for (int i = threadIdx.x; i < count + overrun; i += blockDim.x) buf[i] = 1.f;
}
int ws_guard_selftest(void *ws, size_t bytes, int overrun, cudaStream_t st) {
    if (bytes < 4096) return STREAMBP_E_WORKSPACE;
    Arena a(ws);
    a.guarded = true;
    WsHeader *hdr = reinterpret_cast<WsHeader *>(a.take_bytes(kHeaderBytes));
    float *b0 = a.take<float>(100), *b1 = a.take<float>(77), *b2 = a.take<float>(64);
    (void)b0; (void)b2;
    if (a.size() > bytes) return STREAMBP_E_WORKSPACE;
    SBP_TRY(fill_zero(ws, kHeaderBytes, st));
    SBP_TRY(ws_guards_arm(ws, a.guards, st));
    SBP_LAUNCH(overrun_kernel, 1, 128, 0, st, b1, 77, overrun);
    return ws_guards_check(ws, a.guards, hdr, st);
}

int fill_zero(void *p, size_t bytes, cudaStream_t st) {
    if (bytes == 0 || p == nullptr) return STREAMBP_OK;
    return cuda_ok(cudaMemsetAsync(p, 0, bytes, st)) ? STREAMBP_OK : STREAMBP_E_CUDA;
}

// ---------------------------------------------------------------------------------
// LM head: label count, cross-entropy rows, loss reduction
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
    count_labels_kernel(const int64_t *__restrict__ labels, int64_t T_, int64_t vocab, int64_t ignore, WsHeader *hdr) {
    pdl_enter();
    __shared__ unsigned int cnt;
    if (threadIdx.x == 0) cnt = 0;
    __syncthreads();
    unsigned int mine = 0;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < T_; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t y = labels[t];
        if (y == ignore) continue;
        if (y < 0 || y >= vocab) {
            set_status(hdr, STREAMBP_E_BAD_LABEL, (int)t);
            continue;
        }
        mine++;
    }
    atomicAdd(&cnt, mine);
    __syncthreads();
    if (threadIdx.x == 0 && cnt) atomicAdd(&hdr->n_valid, (unsigned long long)cnt);
}

int count_valid_labels(const int64_t *labels, int64_t T_, int64_t vocab, int64_t ignore, WsHeader *hdr,
                       cudaStream_t st) {
    int blocks = (int)((T_ + 255) / 256);
    if (blocks > 1024) blocks = 1024;
    if (blocks < 1) blocks = 1;
    SBP_LAUNCH(count_labels_kernel, blocks, 256, 0, st, labels, T_, vocab, ignore, hdr);
    return STREAMBP_OK;
}

__global__ void __launch_bounds__(256)
    count_chunk_labels_kernel(const int64_t *__restrict__ labels, int64_t T_, int64_t chunk, int64_t ignore,
                              int *__restrict__ counts) {
    pdl_enter();
    __shared__ int cnt;
    if (threadIdx.x == 0) cnt = 0;
    __syncthreads();
    const int64_t r0 = (int64_t)blockIdx.x * chunk, r1 = min(T_, r0 + chunk);
    int mine = 0;
    for (int64_t t = r0 + threadIdx.x; t < r1; t += blockDim.x) mine += labels[t] != ignore ? 1 : 0;
    atomicAdd(&cnt, mine);
    __syncthreads();
    if (threadIdx.x == 0) counts[blockIdx.x] = cnt;
}
int count_valid_per_chunk(const int64_t *labels, int64_t T_, int64_t chunk, int64_t ignore, int *counts,
                          cudaStream_t st) {
    const int64_t D = (T_ + chunk - 1) / chunk;
    SBP_LAUNCH(count_chunk_labels_kernel, (unsigned)D, 256, 0, st, labels, T_, chunk, ignore, counts);
    return STREAMBP_OK;
}

// one block per logits row: online (max, sum-exp), then dz = (softmax - onehot) / N
template <typename T>
__global__ void __launch_bounds__(1024)
    ce_rows_kernel(const float *z, const int64_t *__restrict__ labels, int64_t V, int64_t ignore,
                   const WsHeader *__restrict__ hdr, T *dz, float *__restrict__ row_loss, const int *gate) {
    pdl_enter();
    __shared__ float red[33];
    __shared__ float zy_s;
    if (gated_off(gate)) return;
    const int64_t row = blockIdx.x;
    const float *zr = z + row * V;
    T *dr = dz + row * V;
    const int64_t y = labels[row];
    const bool valid = (y != ignore) && y >= 0 && y < V;
    const unsigned long long N = hdr->n_valid;
    const bool vec = (V & 3) == 0;
    if (!valid || N == 0) {
        if (vec) {
            const float zero4[4] = {0.f, 0.f, 0.f, 0.f};
            for (int64_t c = threadIdx.x * 4; c < V; c += blockDim.x * 4) store4(dr + c, zero4);
        } else {
            for (int64_t c = threadIdx.x; c < V; c += blockDim.x) dr[c] = from_f32<T>(0.f);
        }
        if (threadIdx.x == 0) row_loss[row] = 0.f;
        return;
    }
    float m = -INFINITY, s = 0.f;
    for (int64_t c = threadIdx.x * 4; c < V; c += blockDim.x * 4) {
        float v[4];
        if (vec && c + 3 < V) {
            const float4 a = *reinterpret_cast<const float4 *>(zr + c);
            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
        } else {
            for (int k = 0; k < 4; k++) v[k] = (c + k < V) ? zr[c + k] : -INFINITY;
        }
        const float mx = fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2], v[3]));
        if (mx > m) {
            s *= __expf(m - mx);
            m = mx;
        }
        s += __expf(v[0] - m) + __expf(v[1] - m) + __expf(v[2] - m) + __expf(v[3] - m);
    }
    const float gm = block_max(m, red);
    s = (m == -INFINITY) ? 0.f : s * __expf(m - gm);
    const float gs = block_sum(s, red);
    if (threadIdx.x == 0) zy_s = zr[y];
    __syncthreads();
    const float lse = gm + logf(gs);
    if (threadIdx.x == 0) row_loss[row] = lse - zy_s;
    const float invN = 1.f / (float)N;
    for (int64_t c = threadIdx.x * 4; c < V; c += blockDim.x * 4) {
        float v[4];
        if (vec && c + 3 < V) {
            const float4 a = *reinterpret_cast<const float4 *>(zr + c);
            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
        } else {
            for (int k = 0; k < 4; k++) v[k] = (c + k < V) ? zr[c + k] : -INFINITY;
        }
        float o[4];
#pragma unroll
        for (int k = 0; k < 4; k++) {
            float p = __expf(v[k] - lse);
            if (c + k == y) p -= 1.f;
            o[k] = p * invN;
        }
        if (vec && c + 3 < V) {
            store4(dr + c, o);       // one 8- or 16-byte store per thread
        } else {
            for (int k = 0; k < 4; k++)
                if (c + k < V) dr[c + k] = from_f32<T>(o[k]);
        }
    }
}

template <typename T>
int ce_rows(const float *z, const int64_t *labels, int64_t rows, int64_t V, int64_t ignore, const WsHeader *hdr,
            T *dz, float *row_loss, cudaStream_t st) {
    if (rows <= 0) return STREAMBP_OK;
    SBP_LAUNCH(ce_rows_kernel<T>, (unsigned)rows, 1024, 0, st, z, labels, V, ignore, hdr, dz, row_loss, call_state().gate);
    return STREAMBP_OK;
}
template int ce_rows<float>(const float *, const int64_t *, int64_t, int64_t, int64_t, const WsHeader *, float *,
                            float *, cudaStream_t);
template int ce_rows<bf16>(const float *, const int64_t *, int64_t, int64_t, int64_t, const WsHeader *, bf16 *,
                           float *, cudaStream_t);

// RL objectives: one block per logits row
template <typename T>
__global__ void __launch_bounds__(1024)
    rl_rows_kernel(const float *z, const int64_t *__restrict__ tokens, int64_t V, int64_t ignore, RlRows rl, int64_t row0,
                   T *dz, float *__restrict__ row_val, const int *gate) {
    pdl_enter();
    __shared__ float red[33];
    __shared__ float zy_s;
    if (gated_off(gate)) return;
    const int64_t row = blockIdx.x, arow = row0 + row;
    const float *zr = z + row * V;
    T *dr = dz + row * V;
    const int64_t y = tokens[row];
    const bool part = (y != ignore) && y >= 0 && y < V;
    const bool vec = (V & 3) == 0;
    if (!part) {
        for (int64_t c = threadIdx.x; c < V; c += blockDim.x) dr[c] = from_f32<T>(0.f);
        if (threadIdx.x == 0) {
            row_val[row] = 0.f;
            if (rl.logp_out) rl.logp_out[arow] = 0.f;
        }
        return;
    }
    float m = -INFINITY, s = 0.f;
    for (int64_t c = threadIdx.x * 4; c < V; c += blockDim.x * 4) {
        float v[4];
        if (vec && c + 3 < V) {
            const float4 a = *reinterpret_cast<const float4 *>(zr + c);
            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
        } else {
            for (int k = 0; k < 4; k++) v[k] = (c + k < V) ? zr[c + k] : -INFINITY;
        }
        const float mx = fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2], v[3]));
        if (mx > m) {
            s *= __expf(m - mx);
            m = mx;
        }
        s += __expf(v[0] - m) + __expf(v[1] - m) + __expf(v[2] - m) + __expf(v[3] - m);
    }
    const float gm = block_max(m, red);
    s = (m == -INFINITY) ? 0.f : s * __expf(m - gm);
    const float gs = block_sum(s, red);
    if (threadIdx.x == 0) zy_s = zr[y];
    __syncthreads();
    const float lse = gm + logf(gs);
    const float logp = zy_s - lse;
    // coefficient c = dL / dlog pi(token) (DPO: before the final sigmoid correction)
    float coef, val;
    if (rl.objective == STREAMBP_OBJ_GRPO) {
        const float w = rl.weight[arow], adv = rl.advantage[arow];
        const float r = expf(logp - rl.logp_old[arow]);
        const float lo = 1.f - rl.clip_eps, hi = 1.f + rl.clip_eps;
        const float unclipped = r * adv, clipped = fminf(fmaxf(r, lo), hi) * adv;
        const bool keeps = (unclipped <= clipped) || (r > lo && r < hi);   // gradient flows through r A
        const float kl = rl.beta * (logp - rl.logp_ref[arow]);
        val = -w * ((keeps ? unclipped : clipped) - kl);
        coef = -w * ((keeps ? unclipped : 0.f) - rl.beta);
    } else {
        const float sgn = rl.weight[arow];
        val = sgn * (logp - rl.logp_ref[arow]);
        coef = rl.beta * sgn;
    }
    if (threadIdx.x == 0) {
        row_val[row] = val;
        if (rl.logp_out) rl.logp_out[arow] = logp;
    }
    for (int64_t c = threadIdx.x * 4; c < V; c += blockDim.x * 4) {
        float v[4];
        if (vec && c + 3 < V) {
            const float4 a = *reinterpret_cast<const float4 *>(zr + c);
            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
        } else {
            for (int k = 0; k < 4; k++) v[k] = (c + k < V) ? zr[c + k] : -INFINITY;
        }
        float o[4];
#pragma unroll
        for (int k = 0; k < 4; k++) {
            float pr = -__expf(v[k] - lse);
            if (c + k == y) pr += 1.f;
            o[k] = coef * pr;
        }
        if (vec && c + 3 < V) {
            store4(dr + c, o);
        } else {
            for (int k = 0; k < 4; k++)
                if (c + k < V) dr[c + k] = from_f32<T>(o[k]);
        }
    }
}

template <typename T>
int rl_rows(const float *z, const int64_t *tokens, int64_t rows, int64_t V, int64_t ignore, const RlRows &rl,
            int64_t row0, T *dz, float *row_val, cudaStream_t st) {
    if (rows <= 0) return STREAMBP_OK;
    SBP_LAUNCH(rl_rows_kernel<T>, (unsigned)rows, 1024, 0, st, z, tokens, V, ignore, rl, row0, dz, row_val,
               call_state().gate);
    return STREAMBP_OK;
}
template int rl_rows<float>(const float *, const int64_t *, int64_t, int64_t, int64_t, const RlRows &, int64_t, float *,
                            float *, cudaStream_t);
template int rl_rows<bf16>(const float *, const int64_t *, int64_t, int64_t, int64_t, const RlRows &, int64_t, bf16 *,
                           float *, cudaStream_t);

__global__ void rl_finalize_kernel(WsHeader *hdr, int objective, float beta, float *loss, float *ell) {
    pdl_enter();
    if (hdr->n_valid == 0) set_status(hdr, STREAMBP_E_NO_VALID_LABELS, 0);
    const double acc = hdr->loss_sum;
    if (objective == STREAMBP_OBJ_GRPO) {
        hdr->factor = 1.f;
        if (loss) *loss = (float)acc;
        if (ell) *ell = 0.f;
    } else {
        // L = -log sigmoid(beta ell) = log(1 + exp(-beta ell)); correction factor sigmoid(beta ell) - 1
        const double x = (double)beta * acc;
        const double sg = 1.0 / (1.0 + exp(-x));
        hdr->factor = hdr->n_valid == 0 ? 0.f : (float)(sg - 1.0);
        if (loss) *loss = hdr->n_valid == 0 ? 0.f : (float)(x > 0 ? log1p(exp(-x)) : -x + log1p(exp(x)));
        if (ell) *ell = (float)acc;
    }
}
int rl_finalize(WsHeader *hdr, int objective, float beta, float *loss, float *ell, cudaStream_t st) {
    SBP_LAUNCH(rl_finalize_kernel, 1, 1, 0, st, hdr, objective, beta, loss, ell);
    return STREAMBP_OK;
}

template <typename T>
__global__ void __launch_bounds__(256) scale_by_factor_kernel(T *p, int64_t n, const WsHeader *hdr) {
    pdl_enter();
    const float f = hdr->factor;
    constexpr int N = Vec<T>::N;
    for (int64_t i0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * N; i0 < n; i0 += (int64_t)gridDim.x * blockDim.x * N) {
        if (i0 + N <= n) {
            Vec<T> a;
            a.load(p + i0);
#pragma unroll
            for (int i = 0; i < N; i++) a.v[i] *= f;
            a.store(p + i0);
        } else {
            for (int64_t i = i0; i < n; i++) p[i] = from_f32<T>(to_f32(p[i]) * f);
        }
    }
}
template <typename T>
int scale_by_factor(T *p, int64_t n, const WsHeader *hdr, cudaStream_t st) {
    if (n <= 0) return STREAMBP_OK;
    int64_t blocks = (n / Vec<T>::N + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (blocks < 1) blocks = 1;
    SBP_LAUNCH(scale_by_factor_kernel<T>, (unsigned)blocks, 256, 0, st, p, n, hdr);
    return STREAMBP_OK;
}
template int scale_by_factor<float>(float *, int64_t, const WsHeader *, cudaStream_t);
template int scale_by_factor<bf16>(bf16 *, int64_t, const WsHeader *, cudaStream_t);

__global__ void __launch_bounds__(1024) loss_accumulate_kernel(const float *__restrict__ row_loss, int64_t rows,
                                                               WsHeader *hdr, const int *gate) {
    pdl_enter();
    __shared__ double red[32];
    if (gated_off(gate)) return;
    double acc = 0.0;
    for (int64_t r = threadIdx.x; r < rows; r += blockDim.x) acc += (double)row_loss[r];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < (int)(blockDim.x >> 5); w++) t += red[w];
        hdr->loss_sum += t;
    }
}
int loss_accumulate(const float *row_loss, int64_t rows, WsHeader *hdr, cudaStream_t st) {
    if (rows <= 0) return STREAMBP_OK;
    SBP_LAUNCH(loss_accumulate_kernel, 1, 1024, 0, st, row_loss, rows, hdr, call_state().gate);
    return STREAMBP_OK;
}

__global__ void loss_finalize_kernel(WsHeader *hdr, float *loss, int64_t *n_valid) {
    pdl_enter();
    const unsigned long long N = hdr->n_valid;
    if (N == 0) {
        set_status(hdr, STREAMBP_E_NO_VALID_LABELS, 0);
        if (loss) *loss = 0.f;
    } else if (loss) {
        *loss = (float)(hdr->loss_sum / (double)N);
    }
    if (n_valid) *n_valid = (int64_t)N;
}
int loss_finalize(WsHeader *hdr, float *loss, int64_t *n_valid, cudaStream_t st) {
    SBP_LAUNCH(loss_finalize_kernel, 1, 1, 0, st, hdr, loss, n_valid);
    return STREAMBP_OK;
}

// ---------------------------------------------------------------------------------
// Embedding
// ---------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
    embedding_gather_kernel(const T *__restrict__ embed, const int64_t *__restrict__ ids, int d, int64_t vocab,
                            T *__restrict__ out, WsHeader *hdr) {
    pdl_enter();
    constexpr int N = Vec<T>::N;
    const int64_t row = blockIdx.x;
    const int64_t id = ids[row];
    const bool ok = id >= 0 && id < vocab;
    if (!ok && threadIdx.x == 0) set_status(hdr, STREAMBP_E_BAD_LABEL, (int)row);
    for (int c = threadIdx.x * N; c < d; c += blockDim.x * N) {
        Vec<T> a;
        if (ok) {
            a.load(embed + id * d + c);
        } else {
#pragma unroll
            for (int i = 0; i < N; i++) a.v[i] = 0.f;
        }
        a.store(out + row * d + c);
    }
}
template <typename T>
int embedding_gather(const T *embed, const int64_t *ids, int64_t rows, int d, int64_t vocab, T *out, WsHeader *hdr,
                     cudaStream_t st) {
    if (rows <= 0) return STREAMBP_OK;
    SBP_LAUNCH(embedding_gather_kernel<T>, (unsigned)rows, 256, 0, st, embed, ids, d, vocab, out, hdr);
    return STREAMBP_OK;
}
template int embedding_gather<float>(const float *, const int64_t *, int64_t, int, int64_t, float *, WsHeader *,
                                     cudaStream_t);
template int embedding_gather<bf16>(const bf16 *, const int64_t *, int64_t, int, int64_t, bf16 *, WsHeader *,
                                    cudaStream_t);

// Deterministic scatter-add: block (column block, token class). A block owns the vocabulary rows whose
// id falls in its class, so every d_embed element is updated by one thread, in token order.
static constexpr int kScatterClasses = 128;
template <typename T>
__global__ void __launch_bounds__(256)
    embedding_scatter_kernel(const T *__restrict__ dx, const int64_t *__restrict__ ids, int64_t rows, int d,
                             int64_t vocab, float *__restrict__ d_embed) {
    pdl_enter();
    const int col = blockIdx.x * 256 + threadIdx.x;
    const int cls = blockIdx.y;
    for (int64_t t = 0; t < rows; t++) {
        const int64_t id = ids[t];
        if (id < 0 || id >= vocab || (int)(id % kScatterClasses) != cls) continue;
        if (col < d) d_embed[id * d + col] += to_f32(dx[t * d + col]);
    }
}
template <typename T>
int embedding_scatter_add(const T *dx, const int64_t *ids, int64_t rows, int d, int64_t vocab, float *d_embed,
                          cudaStream_t st) {
    if (rows <= 0) return STREAMBP_OK;
    dim3 grid((d + 255) / 256, kScatterClasses);
    SBP_LAUNCH(embedding_scatter_kernel<T>, grid, 256, 0, st, dx, ids, rows, d, vocab, d_embed);
    return STREAMBP_OK;
}
template int embedding_scatter_add<float>(const float *, const int64_t *, int64_t, int, int64_t, float *,
                                          cudaStream_t);
template int embedding_scatter_add<bf16>(const bf16 *, const int64_t *, int64_t, int, int64_t, float *, cudaStream_t);

}  // namespace sbp
