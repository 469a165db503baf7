// CNN pieces of the PWL forward pass (Section 3.1: a convolution is a linear operator whose
// matrix dimensions follow from width, height and channels; Section 3: ReLU is already
// piecewise linear, here a 2-segment table in the GEMM epilogue).
//
// A convolution runs as out[M, Cout] = PWL(A[M, K] . W[Cout, K]^T + bias (+ residual)) with
// M = N*Ho*Wo and K = kh*kw*Cin on the tensor-core linear kernel.  This file holds the small
// CUDA-core kernels around it: the zero-padded copies that let a few-channel first layer run as an
// implicit GEMM, the explicit gather (im2col) kept for channel counts the implicit form does not
// take, and the pools.
#include "nm_common.cuh"

namespace {

// A[m][(ky*kw + kx)*Cin + c] = x[n][oy*s - p + ky][ox*s - p + kx][c], zero outside the image.
// Vector path: Cin a multiple of 8, one 16-byte chunk per thread.
template <typename T>
__global__ void __launch_bounds__(256) im2col_vec_kernel(const T* __restrict__ x, T* __restrict__ A, int Nb, int H,
                                                         int W, int Cin, int kh, int kw, int stride, int pad,
                                                         int Ho, int Wo)
{
    // Chunk i of A is (m, ky, kx, c8) = (output pixel, tap, 8 channels), in that order of significance.  A
    // thread visits i, i + step, i + 2 step, ...: its coordinates are decomposed once (the only divisions)
    // and then advanced by the decomposition of `step` with carries, so that the loop is address
    // arithmetic, one 16-byte load and one 16-byte store.
    const int c8n = Cin >> 3;
    const int64_t chunks_per_row = (int64_t)kh * kw * c8n;
    const int64_t total = (int64_t)Nb * Ho * Wo * chunks_per_row;
    const int64_t step = (int64_t)gridDim.x * blockDim.x;
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    int c8, kx, ky, ox, oy, n;
    {
        const int64_t m = i / chunks_per_row;
        const int r = (int)(i - m * chunks_per_row);
        c8 = r % c8n; kx = (r / c8n) % kw; ky = r / (c8n * kw);
        ox = (int)(m % Wo); oy = (int)((m / Wo) % Ho); n = (int)(m / ((int64_t)Wo * Ho));
    }
    int dc8, dkx, dky, dox, doy, dn;
    {
        const int64_t dm = step / chunks_per_row;
        const int dr = (int)(step - dm * chunks_per_row);
        dc8 = dr % c8n; dkx = (dr / c8n) % kw; dky = dr / (c8n * kw);
        dox = (int)(dm % Wo); doy = (int)((dm / Wo) % Ho); dn = (int)(dm / ((int64_t)Wo * Ho));
    }
    for (; i < total; i += step) {
        const int iy = oy * stride - pad + ky, ix = ox * stride - pad + kx;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (iy >= 0 && iy < H && ix >= 0 && ix < W)
            v = __ldg(reinterpret_cast<const uint4*>(x + (((int64_t)n * H + iy) * W + ix) * Cin + c8 * 8));
        *reinterpret_cast<uint4*>(A + i * 8) = v;
        // advance by `step`: every digit gains its share plus the carry of the digit below (each at most once)
        c8 += dc8; if (c8 >= c8n) { c8 -= c8n; ++kx; }
        kx += dkx; if (kx >= kw) { kx -= kw; ++ky; }
        ky += dky; if (ky >= kh) { ky -= kh; ++ox; }
        ox += dox; if (ox >= Wo) { ox -= Wo; ++oy; }
        oy += doy; if (oy >= Ho) { oy -= Ho; ++n; }
        n += dn;
    }
}

// Path for a channel count that is not a multiple of 8 (first layer, Cin = 3): rows padded with zeros
// to Kpad (a multiple of 8).  One thread per 16-byte chunk of A = 8 consecutive k of one output pixel;
// k = (ky*kw + kx)*Cin + c is decomposed once per chunk and stepped with carries, the elements are
// gathered one by one (they are adjacent in x only within a pixel) and leave as one 16-byte store.
template <typename T>
__global__ void __launch_bounds__(256) im2col_scalar_kernel(const T* __restrict__ x, T* __restrict__ A, int Nb, int H,
                                                            int W, int Cin, int kh, int kw, int stride, int pad,
                                                            int Ho, int Wo, int Kpad)
{
    const int K = kh * kw * Cin;
    const int cpr = Kpad >> 3;   // chunks per row
    const int64_t total = (int64_t)Nb * Ho * Wo * cpr;
    const int64_t step = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += step) {
        const int64_t m = i / cpr;
        const int k0 = (int)(i - m * cpr) * 8;
        const int ox = (int)(m % Wo);
        const int oy = (int)((m / Wo) % Ho);
        const int n = (int)(m / ((int64_t)Wo * Ho));
        int c = k0 % Cin, kx = (k0 / Cin) % kw, ky = k0 / (Cin * kw);
        const T* xn = x + (int64_t)n * H * W * Cin;
        const int y0 = oy * stride - pad, x0 = ox * stride - pad;
        T v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int iy = y0 + ky, ix = x0 + kx;
            v[e] = NmType<T>::from_f(0.f);
            if (k0 + e < K && iy >= 0 && iy < H && ix >= 0 && ix < W) v[e] = xn[((int64_t)iy * W + ix) * Cin + c];
            if (++c == Cin) { c = 0; if (++kx == kw) { kx = 0; ++ky; } }
        }
        *reinterpret_cast<uint4*>(A + i * 8) = *reinterpret_cast<const uint4*>(v);
    }
}

// W[Cout][K] -> Wp[Cout][Kpad], zero padded
template <typename T>
__global__ void pad_rows_kernel(const T* __restrict__ w, T* __restrict__ wp, int rows, int K, int Kpad)
{
    const int64_t total = (int64_t)rows * Kpad;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / Kpad;
        const int k = (int)(i - r * Kpad);
        wp[i] = k < K ? w[r * K + k] : NmType<T>::from_f(0.f);
    }
}

// x [N,H,W,Cin] (Cin <= 8) -> xp [N,Hp,Wp,8]: a border of `pad` zero pixels on the top and left (whatever
// remains of Hp, Wp on the bottom and right) and zero channels Cin..7; one 16-byte pixel per thread.
template <typename T>
__global__ void __launch_bounds__(256) pad_input_kernel(const T* __restrict__ x, T* __restrict__ xp, int Nb, int H,
                                                        int W, int Cin, int pad, int Hp, int Wp)
{
    const int64_t total = (int64_t)Nb * Hp * Wp;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int px = (int)(i % Wp), py = (int)((i / Wp) % Hp), n = (int)(i / ((int64_t)Wp * Hp));
        const int ix = px - pad, iy = py - pad;
        T v[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) v[c] = NmType<T>::from_f(0.f);
        if (ix >= 0 && ix < W && iy >= 0 && iy < H) {
            const T* src = x + (((int64_t)n * H + iy) * W + ix) * Cin;
            for (int c = 0; c < Cin; ++c) v[c] = src[c];
        }
        *reinterpret_cast<uint4*>(xp + i * 8) = *reinterpret_cast<const uint4*>(v);
    }
}

// w [Cout,kh,kw,Cin] (kw <= 8, Cin <= 8) -> wp [Cout,kh,8,8], zero where kx >= kw or c >= Cin
template <typename T>
__global__ void pad_weight_kernel(const T* __restrict__ w, T* __restrict__ wp, int Cout, int kh, int kw, int Cin)
{
    const int64_t total = (int64_t)Cout * kh * 64;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int c = (int)(i & 7), kx = (int)((i >> 3) & 7);
        const int64_t r = i >> 6;   // (co, ky)
        wp[i] = (kx < kw && c < Cin) ? w[(r * kw + kx) * Cin + c] : NmType<T>::from_f(0.f);
    }
}

__device__ __forceinline__ float2 unpack2(__half2 v) { return __half22float2(v); }
__device__ __forceinline__ float2 unpack2(__nv_bfloat162 v) { return __bfloat1622float2(v); }
template <typename T> struct Vec2;
template <> struct Vec2<__half> { using type = __half2; static __device__ __forceinline__ __half2 make(float a, float b) { return __floats2half2_rn(a, b); } };
template <> struct Vec2<__nv_bfloat16> { using type = __nv_bfloat162; static __device__ __forceinline__ __nv_bfloat162 make(float a, float b) { return __floats2bfloat162_rn(a, b); } };

// window maximum, padding cells ignored; 8 channels per thread.  With a table (`relu`), the maximum is
// taken in its operator form max(a, b) = b + PWLrelu(a - b), folded over the window in raster order.
template <typename T>
__global__ void __launch_bounds__(256) maxpool_kernel(const T* __restrict__ x, T* __restrict__ y, int Nb, int H, int W,
                                                      int C, int ks, int stride, int pad, int Ho, int Wo,
                                                      const NmTable* __restrict__ relu)
{
    float inv_h = 0.f, off = 0.f, nm1 = 0.f;
    if (relu) { inv_h = relu->inv_h; off = relu->off; nm1 = (float)(relu->n - 1); }
    using V2 = typename Vec2<T>::type;
    const int c8n = C >> 3;
    const int64_t total = (int64_t)Nb * Ho * Wo * c8n;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int c8 = (int)(i % c8n);
        const int64_t m = i / c8n;
        const int ox = (int)(m % Wo), oy = (int)((m / Wo) % Ho), n = (int)(m / ((int64_t)Wo * Ho));
        float best[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) best[j] = -INFINITY;
        bool first = true;
        for (int ky = 0; ky < ks; ++ky) {
            const int iy = oy * stride - pad + ky;
            if (iy < 0 || iy >= H) continue;
            for (int kx = 0; kx < ks; ++kx) {
                const int ix = ox * stride - pad + kx;
                if (ix < 0 || ix >= W) continue;
                const uint4 raw = __ldg(reinterpret_cast<const uint4*>(x + (((int64_t)n * H + iy) * W + ix) * C + c8 * 8));
                const V2* h = reinterpret_cast<const V2*>(&raw);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float2 f = unpack2(h[j]);
                    if (relu && !first) {
                        const float v[2] = {f.x, f.y};
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const float dlt = v[e] - best[2 * j + e];
                            const float2 kb = relu->kb[nm_pwl_index(dlt, inv_h, off, nm1)];
                            best[2 * j + e] += __fmaf_rn(kb.x, dlt, kb.y);
                        }
                    } else if (relu) {
                        best[2 * j] = f.x;
                        best[2 * j + 1] = f.y;
                    } else {
                        best[2 * j] = fmaxf(best[2 * j], f.x);
                        best[2 * j + 1] = fmaxf(best[2 * j + 1], f.y);
                    }
                }
                first = false;
            }
        }
        uint4 out;
        V2* o = reinterpret_cast<V2*>(&out);
#pragma unroll
        for (int j = 0; j < 4; ++j) o[j] = Vec2<T>::make(best[2 * j], best[2 * j + 1]);
        *reinterpret_cast<uint4*>(y + i * 8) = out;
    }
}

// 64 x 64 matrix with `value` on the diagonal: the constant operand of the average pool run as a GEMM
template <typename T>
__global__ void fill_diag_kernel(T* __restrict__ w, float value)
{
    for (int i = threadIdx.x; i < 64 * 64; i += blockDim.x) w[i] = NmType<T>::from_f((i >> 6) == (i & 63) ? value : 0.f);
}

// mean over the HW positions of each image: [N, HW, C] -> [N, C]; 8 channels per thread, fp32 sums
template <typename T>
__global__ void __launch_bounds__(256) avgpool_kernel(const T* __restrict__ x, T* __restrict__ y, int Nb, int HW, int C)
{
    using V2 = typename Vec2<T>::type;
    const int c8n = C >> 3;
    const int64_t total = (int64_t)Nb * c8n;
    const float inv = 1.0f / (float)HW;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int c8 = (int)(i % c8n);
        const int n = (int)(i / c8n);
        float s[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) s[j] = 0.f;
        for (int p = 0; p < HW; ++p) {
            const uint4 raw = __ldg(reinterpret_cast<const uint4*>(x + ((int64_t)n * HW + p) * C + c8 * 8));
            const V2* h = reinterpret_cast<const V2*>(&raw);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 f = unpack2(h[j]);
                s[2 * j] += f.x;
                s[2 * j + 1] += f.y;
            }
        }
        uint4 out;
        V2* o = reinterpret_cast<V2*>(&out);
#pragma unroll
        for (int j = 0; j < 4; ++j) o[j] = Vec2<T>::make(s[2 * j] * inv, s[2 * j + 1] * inv);
        *reinterpret_cast<uint4*>(y + ((int64_t)n * C + c8 * 8)) = out;
    }
}

int grid_for(nm_ctx* ctx, int64_t total)
{
    int64_t want = (total + 255) / 256;
    const int64_t cap = (int64_t)ctx->sm_count * 16;
    return (int)(want < 1 ? 1 : (want > cap ? cap : want));
}

}  // namespace

nm_status nm_launch_im2col(nm_ctx* ctx, const void* x, void* A, nm_dtype dt, int Nb, int H, int W, int Cin, int kh,
                           int kw, int stride, int pad, int Ho, int Wo, int Kpad, cudaStream_t st)
{
    const int64_t M = (int64_t)Nb * Ho * Wo;
    NmLaunchScope scope(ctx, NM_KERNEL_IM2COL, (double)M * Kpad * 2.0 * nm_dtype_size(dt), st);
    if (Cin % 8 == 0) {
        const int64_t total = M * kh * kw * (Cin / 8);
        if (dt == NM_F16)
            im2col_vec_kernel<__half><<<grid_for(ctx, total), 256, 0, st>>>((const __half*)x, (__half*)A, Nb, H, W, Cin, kh, kw, stride, pad, Ho, Wo);
        else
            im2col_vec_kernel<__nv_bfloat16><<<grid_for(ctx, total), 256, 0, st>>>((const __nv_bfloat16*)x, (__nv_bfloat16*)A, Nb, H, W, Cin, kh, kw, stride, pad, Ho, Wo);
    } else {
        const int64_t total = M * (Kpad / 8);
        if (dt == NM_F16)
            im2col_scalar_kernel<__half><<<grid_for(ctx, total), 256, 0, st>>>((const __half*)x, (__half*)A, Nb, H, W, Cin, kh, kw, stride, pad, Ho, Wo, Kpad);
        else
            im2col_scalar_kernel<__nv_bfloat16><<<grid_for(ctx, total), 256, 0, st>>>((const __nv_bfloat16*)x, (__nv_bfloat16*)A, Nb, H, W, Cin, kh, kw, stride, pad, Ho, Wo, Kpad);
    }
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

nm_status nm_launch_pad_input(nm_ctx* ctx, const void* x, void* xp, nm_dtype dt, int Nb, int H, int W, int Cin, int pad,
                              int Hp, int Wp, cudaStream_t st)
{
    const int64_t total = (int64_t)Nb * Hp * Wp;
    NmLaunchScope scope(ctx, NM_KERNEL_IM2COL, ((double)Nb * H * W * Cin + (double)total * 8) * nm_dtype_size(dt), st);
    if (dt == NM_F16) pad_input_kernel<__half><<<grid_for(ctx, total), 256, 0, st>>>((const __half*)x, (__half*)xp, Nb, H, W, Cin, pad, Hp, Wp);
    else pad_input_kernel<__nv_bfloat16><<<grid_for(ctx, total), 256, 0, st>>>((const __nv_bfloat16*)x, (__nv_bfloat16*)xp, Nb, H, W, Cin, pad, Hp, Wp);
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

nm_status nm_launch_pad_weight(nm_ctx* ctx, const void* w, void* wp, nm_dtype dt, int Cout, int kh, int kw, int Cin,
                               cudaStream_t st)
{
    const int64_t total = (int64_t)Cout * kh * 64;
    NmLaunchScope scope(ctx, NM_KERNEL_IM2COL, (double)total * 2.0 * nm_dtype_size(dt), st);
    if (dt == NM_F16) pad_weight_kernel<__half><<<grid_for(ctx, total), 256, 0, st>>>((const __half*)w, (__half*)wp, Cout, kh, kw, Cin);
    else pad_weight_kernel<__nv_bfloat16><<<grid_for(ctx, total), 256, 0, st>>>((const __nv_bfloat16*)w, (__nv_bfloat16*)wp, Cout, kh, kw, Cin);
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

nm_status nm_launch_pad_rows(nm_ctx* ctx, const void* w, void* wp, nm_dtype dt, int rows, int K, int Kpad,
                             cudaStream_t st)
{
    NmLaunchScope scope(ctx, NM_KERNEL_IM2COL, (double)rows * Kpad * 2.0 * nm_dtype_size(dt), st);
    const int64_t total = (int64_t)rows * Kpad;
    if (dt == NM_F16) pad_rows_kernel<__half><<<grid_for(ctx, total), 256, 0, st>>>((const __half*)w, (__half*)wp, rows, K, Kpad);
    else pad_rows_kernel<__nv_bfloat16><<<grid_for(ctx, total), 256, 0, st>>>((const __nv_bfloat16*)w, (__nv_bfloat16*)wp, rows, K, Kpad);
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

nm_status nm_launch_maxpool(nm_ctx* ctx, const void* x, void* y, nm_dtype dt, int Nb, int H, int W, int C, int ks,
                            int stride, int pad, int Ho, int Wo, cudaStream_t st, int relu_slot)
{
    const NmTable* relu = relu_slot == NM_SLOT_NONE ? nullptr : ctx->d_tables + relu_slot;
    const int64_t total = (int64_t)Nb * Ho * Wo * (C / 8);
    NmLaunchScope scope(ctx, NM_KERNEL_POOL, ((double)Nb * H * W * C + (double)Nb * Ho * Wo * C) * nm_dtype_size(dt), st);
    if (dt == NM_F16)
        maxpool_kernel<__half><<<grid_for(ctx, total), 256, 0, st>>>((const __half*)x, (__half*)y, Nb, H, W, C, ks, stride, pad, Ho, Wo, relu);
    else
        maxpool_kernel<__nv_bfloat16><<<grid_for(ctx, total), 256, 0, st>>>((const __nv_bfloat16*)x, (__nv_bfloat16*)y, Nb, H, W, C, ks, stride, pad, Ho, Wo, relu);
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

nm_status nm_launch_fill_diag(nm_ctx* ctx, void* w, nm_dtype dt, float value, cudaStream_t st)
{
    NmLaunchScope scope(ctx, NM_KERNEL_POOL, 64.0 * 64.0 * nm_dtype_size(dt), st);
    if (dt == NM_F16) fill_diag_kernel<__half><<<1, 256, 0, st>>>((__half*)w, value);
    else fill_diag_kernel<__nv_bfloat16><<<1, 256, 0, st>>>((__nv_bfloat16*)w, value);
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

nm_status nm_launch_avgpool(nm_ctx* ctx, const void* x, void* y, nm_dtype dt, int Nb, int HW, int C, cudaStream_t st)
{
    const int64_t total = (int64_t)Nb * (C / 8);
    NmLaunchScope scope(ctx, NM_KERNEL_POOL, ((double)Nb * HW * C + (double)Nb * C) * nm_dtype_size(dt), st);
    if (dt == NM_F16) avgpool_kernel<__half><<<grid_for(ctx, total), 256, 0, st>>>((const __half*)x, (__half*)y, Nb, HW, C);
    else avgpool_kernel<__nv_bfloat16><<<grid_for(ctx, total), 256, 0, st>>>((const __nv_bfloat16*)x, (__nv_bfloat16*)y, Nb, HW, C);
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}
