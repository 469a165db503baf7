// Plain CUDA-core kernels: the fp32 path (whose 1e-4 tolerance rules out
// tensor-core tf32) and the fallback for shapes the tcgen05 kernels do not take.
//   linear:    out = PWL(A.W^T * scale + bias) + residual   (Section 3.1 + 3.2)
//   attention: softmax with PWL exp / PWL reciprocal, final row maximum
#include "nm_common.cuh"

namespace {

template <typename T> struct AccOf { using type = float; };
template <> struct AccOf<int8_t> { using type = int32_t; };

template <typename T> __device__ __forceinline__ typename AccOf<T>::type to_acc(T v) { return NmType<T>::to_f(v); }
template <> __device__ __forceinline__ int32_t to_acc<int8_t>(int8_t v) { return (int32_t)v; }

template <typename OutT> __device__ __forceinline__ void store_out(OutT* p, float y, float) { *p = NmType<OutT>::from_f(y); }
template <> __device__ __forceinline__ void store_out<int8_t>(int8_t* p, float y, float inv) { *p = nm_quant_i8(y, inv); }

template <typename OutT> __device__ __forceinline__ float load_res(const OutT* p) { return NmType<OutT>::to_f(*p); }
template <> __device__ __forceinline__ float load_res<int8_t>(const int8_t*) { return 0.f; }

struct LinArgs {
    int64_t M, N, K, lda, ldw, ldr, ldo;
    const float* bias;
    const void* residual;
    int res_first;       // residual is added before the table instead of after
    const NmTable* tab;  // nullptr: no table
    float a_scale;
    const float* w_scale;
    float inv_out_scale;
    int32_t* acc_dump;
    int32_t* idx_dump;
};

// 64x64 output tile per CTA, 16-deep K slices, each of 256 threads owns a 4x4 block.
template <typename InT, typename OutT>
__global__ void __launch_bounds__(256) linear_simt_kernel(const InT* __restrict__ A, const InT* __restrict__ W,
                                                          OutT* __restrict__ out, LinArgs a)
{
    using Acc = typename AccOf<InT>::type;
    constexpr int BM = 64, BN = 64, BK = 16;
    __shared__ Acc sA[BK][BM + 1];
    __shared__ Acc sB[BK][BN + 1];
    __shared__ float2 s_tab[NM_MAX_SEGMENTS];
    const int tid = threadIdx.x;
    const int64_t m0 = (int64_t)blockIdx.y * BM, n0 = (int64_t)blockIdx.x * BN;
    const int tx = tid & 15, ty = tid >> 4;
    int n_seg = 0;
    float inv_h = 0.f, off = 0.f;
    if (a.tab) {
        n_seg = a.tab->n;
        inv_h = a.tab->inv_h;
        off = a.tab->off;
        for (int i = tid; i < n_seg; i += 256) s_tab[i] = a.tab->kb[i];
    }
    Acc acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0;

    for (int64_t k0 = 0; k0 < a.K; k0 += BK) {
        // 64x16 elements of each operand: 1024 elements, 4 per thread
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            int lin = tid + e * 256;
            int r = lin >> 4, c = lin & 15;
            int64_t gk = k0 + c;
            int64_t gm = m0 + r, gn = n0 + r;
            sA[c][r] = (gm < a.M && gk < a.K) ? to_acc<InT>(A[gm * a.lda + gk]) : (Acc)0;
            sB[c][r] = (gn < a.N && gk < a.K) ? to_acc<InT>(W[gn * a.ldw + gk]) : (Acc)0;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            Acc ra[4], rb[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) ra[i] = sA[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) rb[j] = sB[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if constexpr (sizeof(Acc) == 4 && !__is_same(Acc, float)) acc[i][j] += ra[i] * rb[j];
                    else acc[i][j] = __fmaf_rn(ra[i], rb[j], acc[i][j]);
                }
        }
        __syncthreads();
    }

    const float nm1 = (float)(n_seg - 1);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int64_t gm = m0 + ty * 4 + i;
        if (gm >= a.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int64_t gn = n0 + tx * 4 + j;
            if (gn >= a.N) continue;
            float x;
            const float bj = a.bias ? a.bias[gn] : 0.f;
            if constexpr (__is_same(Acc, int32_t)) {
                if (a.acc_dump) a.acc_dump[gm * a.N + gn] = acc[i][j];
                const float sc = a.a_scale * a.w_scale[gn];
                x = __fmaf_rn((float)acc[i][j], sc, bj);
            } else {
                x = acc[i][j] + bj;
            }
            if (a.residual && a.res_first) x = x + load_res<OutT>((const OutT*)a.residual + gm * a.ldr + gn);
            int s = -1;
            if (a.tab) {
                s = nm_pwl_index(x, inv_h, off, nm1);
                float2 kb = s_tab[s];
                x = __fmaf_rn(kb.x, x, kb.y);
            }
            if (a.idx_dump) a.idx_dump[gm * a.N + gn] = s;
            if (a.residual && !a.res_first) x = x + load_res<OutT>((const OutT*)a.residual + gm * a.ldr + gn);
            store_out<OutT>(out + gm * a.ldo + gn, x, a.inv_out_scale);
        }
    }
}

// ---- attention: one warp per query row --------------------------------------------
//   s_j = scale*<q,k_j>; m = max s; e_j = PWLexp(s_j - m); sigma = sum e; r = PWLrecip(sigma);
//   o = sum_j (e_j*r) v_j
template <typename T>
__global__ void __launch_bounds__(128) attention_simt_kernel(const T* __restrict__ Q, const T* __restrict__ Kp,
                                                             const T* __restrict__ V, T* __restrict__ out,
                                                             int B, int L, int heads, int d, int64_t stride_b,
                                                             int64_t stride_t, float scale,
                                                             const NmTable* __restrict__ t_exp,
                                                             const NmTable* __restrict__ t_rcp)
{
    extern __shared__ float smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float2* s_exp = reinterpret_cast<float2*>(smem);                 // NM_MAX_SEGMENTS
    float* s_q = smem + 2 * NM_MAX_SEGMENTS + warp * d;               // 4 * d
    float* s_e = smem + 2 * NM_MAX_SEGMENTS + 4 * d + (size_t)warp * L;  // 4 * L
    const int n_exp = t_exp->n;
    for (int i = threadIdx.x; i < n_exp; i += blockDim.x) s_exp[i] = t_exp->kb[i];
    const float e_inv_h = t_exp->inv_h, e_off = t_exp->off, e_nm1 = (float)(n_exp - 1);
    __syncthreads();
    const int64_t rows = (int64_t)B * heads * L;
    for (int64_t row = (int64_t)blockIdx.x * 4 + warp; row < rows; row += (int64_t)gridDim.x * 4) {
        const int64_t b = row / ((int64_t)heads * L);
        const int g = (int)((row / L) % heads);
        const int i = (int)(row % L);
        const T* q = Q + b * stride_b + (int64_t)i * stride_t + (int64_t)g * d;
        for (int c = lane; c < d; c += 32) s_q[c] = NmType<T>::to_f(q[c]);
        __syncwarp();
        float m = -INFINITY;
        for (int j = lane; j < L; j += 32) {
            const T* kk = Kp + b * stride_b + (int64_t)j * stride_t + (int64_t)g * d;
            float s = 0.f;
            for (int c = 0; c < d; ++c) s = __fmaf_rn(s_q[c], NmType<T>::to_f(kk[c]), s);
            s *= scale;
            s_e[j] = s;
            m = fmaxf(m, s);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        float sigma = 0.f;
        for (int j = lane; j < L; j += 32) {
            float x = s_e[j] - m;
            int s = nm_pwl_index(x, e_inv_h, e_off, e_nm1);
            float2 kb = s_exp[s];
            float e = __fmaf_rn(kb.x, x, kb.y);
            s_e[j] = e;
            sigma += e;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sigma += __shfl_xor_sync(0xffffffffu, sigma, o);
        const int sr = nm_pwl_index(sigma, t_rcp->inv_h, t_rcp->off, (float)(t_rcp->n - 1));
        const float2 kbr = t_rcp->kb[sr];
        const float r = __fmaf_rn(kbr.x, sigma, kbr.y);
        __syncwarp();
        T* o = out + (b * L + i) * ((int64_t)heads * d) + (int64_t)g * d;
        for (int c = lane; c < d; c += 32) {
            float accv = 0.f;
            for (int j = 0; j < L; ++j) {
                const T* vv = V + b * stride_b + (int64_t)j * stride_t + (int64_t)g * d;
                accv = __fmaf_rn(s_e[j] * r, NmType<T>::to_f(vv[c]), accv);
            }
            o[c] = NmType<T>::from_f(accv);
        }
        __syncwarp();
    }
}

template <typename InT, typename OutT>
nm_status launch_lin(nm_ctx* ctx, const nm_linear_desc* d, cudaStream_t st)
{
    LinArgs a;
    a.M = d->M; a.N = d->N; a.K = d->K; a.lda = d->lda; a.ldw = d->ldw; a.ldr = d->ldr; a.ldo = d->ldo;
    a.bias = d->bias; a.residual = d->residual; a.res_first = d->res_first;
    a.tab = d->slot == NM_SLOT_NONE ? nullptr : ctx->d_tables + d->slot;
    a.a_scale = d->a_scale; a.w_scale = d->w_scale; a.inv_out_scale = d->inv_out_scale;
    a.acc_dump = d->acc_dump; a.idx_dump = d->idx_dump;
    dim3 grid((unsigned)((d->N + 63) / 64), (unsigned)((d->M + 63) / 64));
    if (grid.y > 65535u) return NM_ERR_SHAPE;
    NmLaunchScope scope(ctx, NM_KERNEL_LINEAR_SIMT, 2.0 * (double)d->M * (double)d->N * (double)d->K, st);
    linear_simt_kernel<InT, OutT><<<grid, 256, 0, st>>>((const InT*)d->A, (const InT*)d->W, (OutT*)d->out, a);
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

template <typename T>
nm_status launch_attn(nm_ctx* ctx, const nm_attn_desc* d, cudaStream_t st)
{
    const size_t smem = sizeof(float) * (2 * NM_MAX_SEGMENTS + 4 * (size_t)d->d + 4 * (size_t)d->L);
    if (smem > 200 * 1024) return NM_ERR_UNSUPPORTED;
    auto kern = attention_simt_kernel<T>;
    if (smem > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    const int64_t rows = (int64_t)d->B * d->heads * d->L;
    int64_t want = (rows + 3) / 4;
    int blocks = (int)(want > (int64_t)ctx->sm_count * 16 ? (int64_t)ctx->sm_count * 16 : want);
    NmLaunchScope scope(ctx, NM_KERNEL_ATTENTION_SIMT, 4.0 * (double)d->B * d->heads * (double)d->L * d->L * d->d, st);
    kern<<<blocks, 128, smem, st>>>((const T*)d->Q, (const T*)d->K, (const T*)d->V, (T*)d->out, d->B, d->L,
                                    d->heads, d->d, d->stride_b, d->stride_t, d->scale,
                                    ctx->d_tables + d->exp_slot, ctx->d_tables + d->recip_slot);
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

}  // namespace

nm_status nm_launch_linear_simt(nm_ctx* ctx, const nm_linear_desc* d, cudaStream_t st)
{
    switch (d->in_dtype) {
    case NM_F32: return launch_lin<float, float>(ctx, d, st);
    case NM_BF16: return launch_lin<__nv_bfloat16, __nv_bfloat16>(ctx, d, st);
    case NM_F16: return launch_lin<__half, __half>(ctx, d, st);
    case NM_I8:
        if (d->out_dtype == NM_BF16) return launch_lin<int8_t, __nv_bfloat16>(ctx, d, st);
        if (d->out_dtype == NM_F32) return launch_lin<int8_t, float>(ctx, d, st);
        if (d->out_dtype == NM_I8) return launch_lin<int8_t, int8_t>(ctx, d, st);
        return NM_ERR_UNSUPPORTED;
    }
    return NM_ERR_UNSUPPORTED;
}

nm_status nm_launch_attention_simt(nm_ctx* ctx, const nm_attn_desc* d, cudaStream_t st)
{
    switch (d->dtype) {
    case NM_F32: return launch_attn<float>(ctx, d, st);
    case NM_BF16: return launch_attn<__nv_bfloat16>(ctx, d, st);
    case NM_F16: return launch_attn<__half>(ctx, d, st);
    default: return NM_ERR_UNSUPPORTED;
    }
}
