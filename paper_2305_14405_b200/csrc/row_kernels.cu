// HBM-bound kernels of the PWL forward pass: element-wise table evaluation,
// LayerNorm with PWL rsqrt, and int8 quantisation.  One read and one write per
// element, 128-bit accesses, no staging through shared memory needed.
#include <string.h>

#include "nm_common.cuh"

namespace {

template <typename T, int VEC> struct Pack {
    T v[VEC];
};

template <typename T> struct VecOf { static constexpr int N = 16 / sizeof(T); };

template <typename T>
__device__ __forceinline__ void load16(const T* p, float* f)
{
    constexpr int N = VecOf<T>::N;
    uint4 raw = *reinterpret_cast<const uint4*>(p);
    const T* e = reinterpret_cast<const T*>(&raw);
#pragma unroll
    for (int i = 0; i < N; ++i) f[i] = NmType<T>::to_f(e[i]);
}

template <typename T>
__device__ __forceinline__ void store16(T* p, const float* f)
{
    constexpr int N = VecOf<T>::N;
    uint4 raw;
    T* e = reinterpret_cast<T*>(&raw);
#pragma unroll
    for (int i = 0; i < N; ++i) e[i] = NmType<T>::from_f(f[i]);
    *reinterpret_cast<uint4*>(p) = raw;
}

// ---- y = k[s]*x + b[s] element-wise (Section 3.2: S, then Y = X.K + B) ----------
template <typename T>
__global__ void __launch_bounds__(256) pwl_apply_kernel(const NmTable* __restrict__ tab, const T* __restrict__ x,
                                                        T* __restrict__ y, int64_t count,
                                                        int32_t* __restrict__ idx_out)
{
    extern __shared__ float2 rep[];
    const int n = tab->n;
    const float inv_h = tab->inv_h, off = tab->off, nm1 = (float)(n - 1);
    nm_table_replicate(rep, tab, n, threadIdx.x, blockDim.x);
    __syncthreads();
    const int lane = threadIdx.x & 31;
    constexpr int N = VecOf<T>::N;
    const int64_t nvec = count / N;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < nvec; v += stride) {
        float f[N];
        int s[N];
        load16<T>(x + v * N, f);
#pragma unroll
        for (int i = 0; i < N; ++i) f[i] = nm_pwl_eval_rep(rep, lane, f[i], inv_h, off, nm1, &s[i]);
        store16<T>(y + v * N, f);
        if (idx_out) {
#pragma unroll
            for (int i = 0; i < N; i += 4)
                *reinterpret_cast<int4*>(idx_out + v * N + i) = make_int4(s[i], s[i + 1], s[i + 2], s[i + 3]);
        }
    }
    // ragged tail (count not a multiple of the vector width)
    if (blockIdx.x == 0) {
        for (int64_t i = nvec * N + threadIdx.x; i < count; i += blockDim.x) {
            int s;
            float r = nm_pwl_eval_rep(rep, lane, NmType<T>::to_f(x[i]), inv_h, off, nm1, &s);
            y[i] = NmType<T>::from_f(r);
            if (idx_out) idx_out[i] = s;
        }
    }
}

// ---- LayerNorm with PWL rsqrt: one warp per row, the row kept in registers ------
//   mu = mean(z); v = mean((z-mu)^2); r = PWL_rsqrt(v + eps); y = (z-mu)*r*gamma + beta
// GB_REGS: the lane's gamma and beta values stay in registers for all of the warp's rows (2 x ITERS x N
// registers: rows up to 32 x 3 vectors, two blocks per SM).  Otherwise they are fetched per row through L1,
// which then carries four times the bytes of the row itself and ~700 exposed cycles per row.
template <typename T, int ITERS, bool GB_REGS>
__global__ void __launch_bounds__(256, GB_REGS ? 2 : 1) layernorm_kernel(const NmTable* __restrict__ tab,
                                                        const NmTable* __restrict__ tab2, const T* __restrict__ x,
                                                        const float* __restrict__ gamma,
                                                        const float* __restrict__ beta, T* __restrict__ y,
                                                        int64_t rows, int H, float eps, int8_t* __restrict__ q,
                                                        float q_inv_scale)
{
    // A warp walks over rows with a grid-wide stride; the raw 16-byte vectors of its NEXT row are
    // already in flight while the current row is reduced and written, so every SM keeps several
    // rows per warp outstanding instead of one short-lived row.
    constexpr int N = VecOf<T>::N;
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int nvec = H / N;  // H is a multiple of N
    const float inv_h = tab->inv_h, off = tab->off, nm1 = (float)(tab->n - 1);
    nm_grid_launch_dependents();   // the next kernel may start its set-up
    nm_grid_dependency_wait();     // x comes from the previous kernel
    uint4 nxt[ITERS];
    if (warp0 < rows) {
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
            const int v = it * 32 + lane;
            if (v < nvec) nxt[it] = *reinterpret_cast<const uint4*>(x + warp0 * H + v * N);
        }
    }
    float rg[GB_REGS ? ITERS : 1][N], rb[GB_REGS ? ITERS : 1][N];
    if constexpr (GB_REGS) {
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
            const int v = it * 32 + lane;
            if (v < nvec) {
#pragma unroll
                for (int i = 0; i < N; i += 4) {
                    *reinterpret_cast<float4*>(&rg[it][i]) = __ldg(reinterpret_cast<const float4*>(gamma + v * N + i));
                    *reinterpret_cast<float4*>(&rb[it][i]) = __ldg(reinterpret_cast<const float4*>(beta + v * N + i));
                }
            }
        }
    }
    for (int64_t row = warp0; row < rows; row += nwarps) {
        float f[ITERS][N];
        float sum = 0.f;
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
            const int v = it * 32 + lane;
            if (v < nvec) {
                const T* e = reinterpret_cast<const T*>(&nxt[it]);
#pragma unroll
                for (int i = 0; i < N; ++i) {
                    f[it][i] = NmType<T>::to_f(e[i]);
                    sum += f[it][i];
                }
            }
        }
        const int64_t nrow = row + nwarps;
        if (nrow < rows) {
#pragma unroll
            for (int it = 0; it < ITERS; ++it) {
                const int v = it * 32 + lane;
                if (v < nvec) nxt[it] = *reinterpret_cast<const uint4*>(x + nrow * H + v * N);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        const float mu = sum / (float)H;
        float sq = 0.f;
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
            const int v = it * 32 + lane;
            if (v < nvec) {
#pragma unroll
                for (int i = 0; i < N; ++i) {
                    const float dlt = f[it][i] - mu;
                    f[it][i] = dlt;
                    sq = __fmaf_rn(dlt, dlt, sq);
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
        const float var = sq / (float)H + eps;
        const int s = nm_pwl_index(var, inv_h, off, nm1);
        const float2 kb = tab->kb[s];
        float r = __fmaf_rn(kb.x, var, kb.y);
        if (tab2) {   // two-table form: `tab` gave sqrt(v + eps), `tab2` takes its reciprocal
            const int s2 = nm_pwl_index(r, tab2->inv_h, tab2->off, (float)(tab2->n - 1));
            const float2 kb2 = tab2->kb[s2];
            r = __fmaf_rn(kb2.x, r, kb2.y);
        }
        T* yr = y + row * H;
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
            const int v = it * 32 + lane;
            if (v < nvec) {
                float g[N], b[N];
                if constexpr (GB_REGS) {
#pragma unroll
                    for (int i = 0; i < N; ++i) {
                        g[i] = rg[it][i];
                        b[i] = rb[it][i];
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < N; i += 4) {
                        *reinterpret_cast<float4*>(&g[i]) = __ldg(reinterpret_cast<const float4*>(gamma + v * N + i));
                        *reinterpret_cast<float4*>(&b[i]) = __ldg(reinterpret_cast<const float4*>(beta + v * N + i));
                    }
                }
#pragma unroll
                for (int i = 0; i < N; ++i) f[it][i] = __fmaf_rn(f[it][i] * r, g[i], b[i]);
                store16<T>(yr + v * N, f[it]);
                if (q) {   // the int8 code of the value as stored (rounded to T first), for the next int8 GEMM
                    int8_t code[N];
#pragma unroll
                    for (int i = 0; i < N; ++i)
                        code[i] = nm_quant_i8(NmType<T>::to_f(NmType<T>::from_f(f[it][i])), q_inv_scale);
                    int8_t* qp = q + row * H + v * N;
                    if constexpr (N == 8) *reinterpret_cast<uint2*>(qp) = *reinterpret_cast<const uint2*>(code);
                    else *reinterpret_cast<uint32_t*>(qp) = *reinterpret_cast<const uint32_t*>(code);
                }
            }
        }
    }
}

// ---- symmetric int8 quantisation with a static scale -----------------------------
template <typename T>
__global__ void __launch_bounds__(256) quantize_kernel(const T* __restrict__ x, int64_t count, float inv_scale,
                                                       int8_t* __restrict__ q)
{
    // 16 elements per thread: one or more 16-byte loads, one 16-byte store
    const int64_t nchunk = count / 16;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    constexpr int N = VecOf<T>::N;
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < nchunk; c += stride) {
        float f[16];
#pragma unroll
        for (int i = 0; i < 16; i += N) load16<T>(x + c * 16 + i, f + i);
        uint4 raw;
        int8_t* e = reinterpret_cast<int8_t*>(&raw);
#pragma unroll
        for (int i = 0; i < 16; ++i) e[i] = nm_quant_i8(f[i], inv_scale);
        *reinterpret_cast<uint4*>(q + c * 16) = raw;
    }
    if (blockIdx.x == 0) {
        for (int64_t i = nchunk * 16 + threadIdx.x; i < count; i += blockDim.x)
            q[i] = nm_quant_i8(NmType<T>::to_f(x[i]), inv_scale);
    }
}

// One warp waits on a barrier that nothing ever arrives on: exercises the bounded wait every
// tensor-core kernel relies on.  The wait gives up after `limit_cycles`, records the timeout in
// the status word and the kernel returns normally (no trap, the context stays usable).
__global__ void wait_selftest_kernel(int* status, long long limit_cycles, int* reached_end)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        nm_mbar_init(&bar, 1);
        nm_fence_barrier_init();
    }
    __syncthreads();
    int ok = 1;
    if (threadIdx.x == 0) ok = nm_mbar_wait_limit(&bar, 0, &abort_flag, status, limit_cycles) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    __syncthreads();
    if (threadIdx.x == 0) *reached_end = ok ? 2 : 1;   // 1: gave up and fell through to the common exit
}

template <typename T>
nm_status launch_ln(nm_ctx* ctx, const NmTable* tab, const NmTable* tab2, const void* x, const float* gamma, const float* beta, void* y,
                    int64_t rows, int H, float eps, int8_t* q, float q_inv_scale, cudaStream_t st)
{
    constexpr int N = VecOf<T>::N;
    const int nvec = H / N;
    const int iters = (nvec + 31) / 32;
    const int threads = 256;
    // Tensors that fit the L2 (the encoder's: 16384 x 768 is 25 MB) are latency-bound: gamma and beta in registers,
    // one resident wave of 2 blocks per SM, 9.9 instead of 13.3 us for that shape.  Tensors far beyond the L2 are
    // bandwidth-bound and want more warps per SM: the per-row fetch of gamma and beta, 6 blocks of 8 warps per SM
    // (5.5 instead of 4.9 TB/s at 2^19 x 768).
    const bool small = (double)rows * H * sizeof(T) <= 48e6 && iters <= 3;
    int64_t blocks = (rows + 7) / 8;
 NmLaunchScope scope(ctx, NM_KERNEL_LAYERNORM, 2.0 * (double)rows * H * sizeof(T), st);
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(threads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = ctx->pdl ? 1 : 0;
    const T* xt = (const T*)x;
    T* yt = (T*)y;
#define NM_LN_CASE(I, GB)                                                                                     \
    do {                                                                                                      \
        static int resident = 0;   /* blocks per SM that this instantiation's registers allow */              \
        if (GB && resident == 0 &&                                                                            \
            (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, layernorm_kernel<T, I, GB>, threads, 0) != \
                 cudaSuccess || resident < 1))                                                                \
            resident = 2;                                                                                     \
        const int64_t cap = (int64_t)ctx->sm_count * (GB ? resident : 6);                                     \
        cfg.gridDim = dim3((unsigned)(blocks > cap ? cap : blocks));                                          \
        cudaLaunchKernelEx(&cfg, layernorm_kernel<T, I, GB>, tab, tab2, xt, gamma, beta, yt, rows, H, eps, q,  \
                           q_inv_scale);                                                                      \
    } while (0)
    if (small && iters <= 1) NM_LN_CASE(1, true);
    else if (small && iters <= 2) NM_LN_CASE(2, true);
    else if (small && iters <= 3) NM_LN_CASE(3, true);
    else if (iters <= 1) NM_LN_CASE(1, false);
    else if (iters <= 2) NM_LN_CASE(2, false);
    else if (iters <= 3) NM_LN_CASE(3, false);
    else if (iters <= 4) NM_LN_CASE(4, false);
    else if (iters <= 8) NM_LN_CASE(8, false);
    else if (iters <= 16) NM_LN_CASE(16, false);
    else return NM_ERR_UNSUPPORTED;
#undef NM_LN_CASE
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

}  // namespace

nm_status nm_launch_pwl_apply(nm_ctx* ctx, int slot, const void* x, void* y, int64_t count, nm_dtype dtype,
                              int32_t* idx_out, cudaStream_t st)
{
    const NmTable* tab = ctx->d_tables + slot;
    const int n = ctx->h_tables[slot].n;
    const size_t smem = (size_t)n * 32 * sizeof(float2);
    const int threads = 256;
    int64_t want = (count / 8 + threads - 1) / threads;
    int blocks = (int)(want < 1 ? 1 : (want > (int64_t)ctx->sm_count * 8 ? (int64_t)ctx->sm_count * 8 : want));
    NmLaunchScope scope(ctx, NM_KERNEL_PWL_APPLY, 2.0 * (double)count * nm_dtype_size(dtype), st);
    switch (dtype) {
    case NM_F32:
        cudaFuncSetAttribute(pwl_apply_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 65536);
        pwl_apply_kernel<float><<<blocks, threads, smem, st>>>(tab, (const float*)x, (float*)y, count, idx_out);
        break;
    case NM_BF16:
        cudaFuncSetAttribute(pwl_apply_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 65536);
        pwl_apply_kernel<__nv_bfloat16>
            <<<blocks, threads, smem, st>>>(tab, (const __nv_bfloat16*)x, (__nv_bfloat16*)y, count, idx_out);
        break;
    case NM_F16:
        cudaFuncSetAttribute(pwl_apply_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, 65536);
        pwl_apply_kernel<__half><<<blocks, threads, smem, st>>>(tab, (const __half*)x, (__half*)y, count, idx_out);
        break;
    default: return NM_ERR_UNSUPPORTED;
    }
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

nm_status nm_launch_layernorm(nm_ctx* ctx, const void* x, const float* gamma, const float* beta, void* y,
                              int64_t rows, int32_t H, float eps, int32_t slot, int32_t slot2, nm_dtype dtype,
                              cudaStream_t st, int8_t* q, float q_inv_scale)
{
    const NmTable* tab = ctx->d_tables + slot;
    const NmTable* tab2 = slot2 == NM_SLOT_NONE ? nullptr : ctx->d_tables + slot2;
    switch (dtype) {
    case NM_F32: return launch_ln<float>(ctx, tab, tab2, x, gamma, beta, y, rows, H, eps, q, q_inv_scale, st);
    case NM_BF16: return launch_ln<__nv_bfloat16>(ctx, tab, tab2, x, gamma, beta, y, rows, H, eps, q, q_inv_scale, st);
    case NM_F16: return launch_ln<__half>(ctx, tab, tab2, x, gamma, beta, y, rows, H, eps, q, q_inv_scale, st);
    default: return NM_ERR_UNSUPPORTED;
    }
}

nm_status nm_launch_wait_selftest(nm_ctx* ctx, long long limit_cycles, cudaStream_t st)
{
    // the second word of the status allocation would be cleaner; the kernel only needs one scratch int,
    // for which the (unused) padding of table slot NM_NUM_SLOTS-1 serves
    int* scratch = &ctx->d_tables[NM_NUM_SLOTS - 1].pad[0];
    NmLaunchScope scope(ctx, NM_KERNEL_PWL_APPLY, 0.0, st);
    wait_selftest_kernel<<<1, 32, 0, st>>>(ctx->d_status, limit_cycles, scratch);
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

nm_status nm_launch_quantize(nm_ctx* ctx, const void* x, nm_dtype dtype, int64_t count, float inv_scale,
                             int8_t* q, cudaStream_t st)
{
    const int threads = 256;
    int64_t want = (count / 16 + threads - 1) / threads;
    int blocks = (int)(want < 1 ? 1 : (want > (int64_t)ctx->sm_count * 16 ? (int64_t)ctx->sm_count * 16 : want));
    NmLaunchScope scope(ctx, NM_KERNEL_QUANTIZE, (double)count * (nm_dtype_size(dtype) + 1), st);
    switch (dtype) {
    case NM_F32: quantize_kernel<float><<<blocks, threads, 0, st>>>((const float*)x, count, inv_scale, q); break;
    case NM_BF16:
        quantize_kernel<__nv_bfloat16><<<blocks, threads, 0, st>>>((const __nv_bfloat16*)x, count, inv_scale, q);
        break;
    case NM_F16: quantize_kernel<__half><<<blocks, threads, 0, st>>>((const __half*)x, count, inv_scale, q); break;
    default: return NM_ERR_UNSUPPORTED;
    }
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}
