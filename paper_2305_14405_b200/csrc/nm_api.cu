// C ABI of the library: context, table construction and loading, argument
// validation, kernel selection, and the encoder-layer sequencing.  All arithmetic
// of the forward pass happens in the kernels this file launches.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "nm_common.cuh"

// Scratch for nm_encoder_layer_static: a fixed array in the library's own device image.  Every
// GPU that loads the library carries these NM_STATIC_WS_BYTES until the process exits.
// In host code the name `nm_static_ws` is only a handle for the runtime, not a device address:
// the address a kernel may use is the one cudaGetSymbolAddress returns, per device.  nm_ctx_create
// resolves it (with the context's device current) and keeps it in the context.
static __device__ __align__(256) unsigned char nm_static_ws[NM_STATIC_WS_BYTES];

namespace {

bool valid_slot(int s) { return s >= 0 && s < NM_NUM_SLOTS; }

nm_status need_table(nm_ctx* ctx, int slot)
{
    if (!valid_slot(slot)) return NM_ERR_INVALID_ARG;
    if (!ctx->h_tables[slot].loaded) return NM_ERR_NO_TABLE;
    return NM_OK;
}

double exact_fn(int func, double x)
{
    switch (func) {
    case NM_FUNC_GELU: return 0.5 * x * (1.0 + erf(x / sqrt(2.0)));
    case NM_FUNC_EXP: return exp(x);
    case NM_FUNC_RECIP: return 1.0 / x;
    case NM_FUNC_RSQRT: return 1.0 / sqrt(x);
    case NM_FUNC_RELU: return x > 0.0 ? x : 0.0;
    case NM_FUNC_SQRT: return sqrt(x);
    case NM_FUNC_IDENTITY: return x;
    }
    return NAN;
}

// F with F' = f, for the segment mean of Algorithm 3
double antiderivative_fn(int func, double x)
{
    switch (func) {
    case NM_FUNC_GELU: {
        const double Phi = 0.5 * (1.0 + erf(x / sqrt(2.0)));
        const double phi = exp(-0.5 * x * x) / sqrt(2.0 * 3.14159265358979323846);
        return 0.5 * (x * x - 1.0) * Phi + 0.5 * x * phi;
    }
    case NM_FUNC_EXP: return exp(x);
    case NM_FUNC_RECIP: return log(x);
    case NM_FUNC_RSQRT: return 2.0 * sqrt(x);
    case NM_FUNC_RELU: return x > 0.0 ? 0.5 * x * x : 0.0;
    case NM_FUNC_SQRT: return (2.0 / 3.0) * x * sqrt(x);
    case NM_FUNC_IDENTITY: return 0.5 * x * x;
    }
    return NAN;
}

}  // namespace

extern "C" {

const char* nm_status_string(nm_status s)
{
    switch (s) {
    case NM_OK: return "NM_OK";
    case NM_ERR_INVALID_ARG: return "NM_ERR_INVALID_ARG";
    case NM_ERR_SHAPE: return "NM_ERR_SHAPE";
    case NM_ERR_ALIGNMENT: return "NM_ERR_ALIGNMENT";
    case NM_ERR_NO_TABLE: return "NM_ERR_NO_TABLE";
    case NM_ERR_UNSUPPORTED: return "NM_ERR_UNSUPPORTED";
    case NM_ERR_CUDA: return "NM_ERR_CUDA";
    case NM_ERR_TIMEOUT: return "NM_ERR_TIMEOUT";
    case NM_ERR_WORKSPACE: return "NM_ERR_WORKSPACE";
    }
    return "NM_ERR_UNKNOWN";
}

nm_status nm_ctx_create(nm_ctx** out, int device)
{
    if (!out) return NM_ERR_INVALID_ARG;
    *out = nullptr;
    NM_CUDA_TRY(cudaSetDevice(device));
    nm_ctx* ctx = new (std::nothrow) nm_ctx();
    if (!ctx) return NM_ERR_CUDA;
    memset(ctx, 0, sizeof(*ctx));
    ctx->device = device;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete ctx; return NM_ERR_CUDA; }
    ctx->sm_count = prop.multiProcessorCount;
    if (prop.major != 10) { delete ctx; return NM_ERR_UNSUPPORTED; }  // kernels are built for sm_100a only
    if (cudaMalloc(&ctx->d_tables, sizeof(NmTable) * NM_NUM_SLOTS) != cudaSuccess) { delete ctx; return NM_ERR_CUDA; }
    if (cudaMalloc(&ctx->d_status, sizeof(int)) != cudaSuccess) { cudaFree(ctx->d_tables); delete ctx; return NM_ERR_CUDA; }
    if (cudaMalloc(&ctx->d_pool_w, 64 * 64 * 2) != cudaSuccess) { cudaFree(ctx->d_tables); cudaFree(ctx->d_status); delete ctx; return NM_ERR_CUDA; }
    cudaMemset(ctx->d_tables, 0, sizeof(NmTable) * NM_NUM_SLOTS);
    cudaMemset(ctx->d_status, 0, sizeof(int));
    cudaDriverEntryPointQueryResult qres;
    void* fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn) {
        cudaFree(ctx->d_tables); cudaFree(ctx->d_status); cudaFree(ctx->d_pool_w); delete ctx;
        return NM_ERR_CUDA;
    }
    ctx->encode_tiled = fn;
    {
        // device address of the library's fixed scratch array on THIS device (the device is current here);
        // a failure is reported by nm_encoder_layer_static, the only call that needs it
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, nm_static_ws) != cudaSuccess) { p = nullptr; (void)cudaGetLastError(); }
        ctx->static_ws = p;
    }
    {
        const char* e = getenv("NM_PDL");   // NM_PDL=0 turns programmatic dependent launch off
        ctx->pdl = (e && e[0] == '0') ? 0 : 1;
        e = getenv("NM_ATTN_RESIDENT");     // NM_ATTN_RESIDENT=1: algo 0 picks the resident-score attention kernel
        ctx->attn_resident = (e && e[0] == '1') ? 1 : 0;
    }
    ctx->prof = new (std::nothrow) NmProfRecord[NM_PROF_MAX];
    if (!ctx->prof) { cudaFree(ctx->d_tables); cudaFree(ctx->d_status); cudaFree(ctx->d_pool_w); delete ctx; return NM_ERR_CUDA; }
    *out = ctx;
    return NM_OK;
}

nm_status nm_ctx_destroy(nm_ctx* ctx)
{
    if (!ctx) return NM_ERR_INVALID_ARG;
    for (int i = 0; i < ctx->prof_created; ++i) {
        cudaEventDestroy(ctx->prof[i].start);
        cudaEventDestroy(ctx->prof[i].stop);
    }
    delete[] ctx->prof;
    cudaFree(ctx->d_tables);
    cudaFree(ctx->d_status);
    cudaFree(ctx->d_pool_w);
    delete ctx;
    return NM_OK;
}

nm_status nm_ctx_poll_status(nm_ctx* ctx, int* device_status, void* stream)
{
    if (!ctx || !device_status) return NM_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    int v = 0;
    NM_CUDA_TRY(cudaMemcpyAsync(&v, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
    NM_CUDA_TRY(cudaStreamSynchronize(st));
    if (v != 0) {
        NM_CUDA_TRY(cudaMemsetAsync(ctx->d_status, 0, sizeof(int), st));
        NM_CUDA_TRY(cudaStreamSynchronize(st));
    }
    *device_status = v;
    return NM_OK;
}

int64_t nm_ctx_launch_count(nm_ctx* ctx, int reset)
{
    if (!ctx) return -1;
    int64_t v = ctx->launches;
    if (reset) ctx->launches = 0;
    return v;
}

nm_status nm_ctx_profile_enable(nm_ctx* ctx, int on)
{
    if (!ctx) return NM_ERR_INVALID_ARG;
    ctx->profiling = on ? 1 : 0;
    ctx->prof_count = 0;
    return NM_OK;
}

nm_status nm_ctx_profile_read(nm_ctx* ctx, int kind, int64_t* launches, double* total_ms, double* total_work)
{
    if (!ctx || !launches || !total_ms || !total_work) return NM_ERR_INVALID_ARG;
    if (kind < 0 || kind >= NM_NUM_KERNEL_KINDS) return NM_ERR_INVALID_ARG;
    int64_t n = 0;
    double ms = 0.0, work = 0.0;
    for (int i = 0; i < ctx->prof_count; ++i) {
        const NmProfRecord* r = &ctx->prof[i];
        if (r->kind != kind) continue;
        NM_CUDA_TRY(cudaEventSynchronize(r->stop));
        float t = 0.f;
        NM_CUDA_TRY(cudaEventElapsedTime(&t, r->start, r->stop));
        ms += (double)t;
        work += r->work;
        ++n;
    }
    *launches = n;
    *total_ms = ms;
    *total_work = work;
    return NM_OK;
}

nm_status nm_pwl_table_build(int func, int n, float x_min, float x_max, float* k_host, float* b_host)
{
    if (!k_host || !b_host) return NM_ERR_INVALID_ARG;
    if (func < NM_FUNC_GELU || func > NM_FUNC_IDENTITY) return NM_ERR_INVALID_ARG;
    if (n < 1 || n > NM_MAX_SEGMENTS || !(x_max > x_min)) return NM_ERR_SHAPE;
    const double lo = (double)x_min, hi = (double)x_max;
    const double h = (hi - lo) / (double)n;
    for (int i = 0; i < n; ++i) {
        const double x0 = lo + (double)i * h, x1 = lo + (double)(i + 1) * h;
        const double f0 = exact_fn(func, x0), f1 = exact_fn(func, x1);
        const double k = (f1 - f0) / (x1 - x0);
        k_host[i] = (float)k;
        b_host[i] = (float)(f0 - k * x0);
    }
    return NM_OK;
}

nm_status nm_pwl_table_build_elastic(int func, float r_min, float r_max, float dLx, float dK_th, int bias_correct,
                                     float e_th, int* n_cells_out, int* n_segments_out, float* k_host, float* b_host)
{
    if (!n_cells_out || !n_segments_out || !k_host || !b_host) return NM_ERR_INVALID_ARG;
    if (func < NM_FUNC_GELU || func > NM_FUNC_IDENTITY) return NM_ERR_INVALID_ARG;
    if (!(r_max > r_min) || !(dLx > 0.f) || dK_th < 0.f || e_th < 0.f) return NM_ERR_SHAPE;
    const double lo = (double)r_min, hi = (double)r_max, step = (double)dLx;
    const double cells = (hi - lo) / step;
    const int n = (int)llround(cells);
    if (n < 1 || n > NM_MAX_SEGMENTS || fabs(cells - (double)n) > 1e-6 * cells) return NM_ERR_SHAPE;
    // Algorithm 2: start cells of the kept segments
    int start[NM_MAX_SEGMENTS + 1];
    int nseg = 0;
    start[nseg++] = 0;
    auto cell_slope = [&](int c) {
        const double x0 = lo + (double)c * step, x1 = lo + (double)(c + 1) * step;
        return (exact_fn(func, x1) - exact_fn(func, x0)) / step;
    };
    double kref = cell_slope(0);
    for (int c = 1; c < n; ++c) {
        const double kc = cell_slope(c);
        if (fabs(kc - kref) > (double)dK_th) {
            start[nseg++] = c;
            kref = kc;
        }
    }
    start[nseg] = n;
    // Algorithm 3 per kept segment, replicated over its primary cells
    for (int s = 0; s < nseg; ++s) {
        const double xa = lo + (double)start[s] * step;
        const double xb = (start[s + 1] == n) ? hi : lo + (double)start[s + 1] * step;
        const double fa = exact_fn(func, xa), fb = exact_fn(func, xb);
        const double k = (fb - fa) / (xb - xa);
        double b = fa - k * xa;
        if (bias_correct) {
            const double dE = (antiderivative_fn(func, xb) - antiderivative_fn(func, xa)) / (xb - xa) - 0.5 * (fa + fb);
            if (fabs(dE) > (double)e_th) b += dE;
        }
        for (int c = start[s]; c < start[s + 1]; ++c) {
            k_host[c] = (float)k;
            b_host[c] = (float)b;
        }
    }
    *n_cells_out = n;
    *n_segments_out = nseg;
    return NM_OK;
}

nm_status nm_pwl_table_load(nm_ctx* ctx, int slot, int n, float x_min, float x_max, const float* k_host,
                            const float* b_host)
{
    if (!ctx || !k_host || !b_host || !valid_slot(slot)) return NM_ERR_INVALID_ARG;
    if (n < 1 || n > NM_MAX_SEGMENTS || !(x_max > x_min)) return NM_ERR_SHAPE;
    NmTable* t = &ctx->h_tables[slot];
    memset(t, 0, sizeof(*t));
    const double span = (double)x_max - (double)x_min;
    t->n = n;
    t->inv_h = (float)((double)n / span);
    t->off = (float)(-(double)x_min * (double)n / span);
    t->x_min = x_min;
    t->x_max = x_max;
    t->loaded = 1;
    for (int i = 0; i < n; ++i) t->kb[i] = make_float2(k_host[i], b_host[i]);
    NM_CUDA_TRY(cudaSetDevice(ctx->device));
    NM_CUDA_TRY(cudaMemcpy(ctx->d_tables + slot, t, sizeof(NmTable), cudaMemcpyHostToDevice));
    return NM_OK;
}

nm_status nm_pwl_apply(nm_ctx* ctx, int slot, const void* x, void* y, int64_t count, nm_dtype dtype,
                       int32_t* idx_out, void* stream)
{
    if (!ctx) return NM_ERR_INVALID_ARG;
    if (count < 0) return NM_ERR_SHAPE;
    nm_status s = need_table(ctx, slot);
    if (s != NM_OK) return s;
    if (count == 0) return NM_OK;
    if (!x || !y) return NM_ERR_INVALID_ARG;
    if (!nm_aligned16(x) || !nm_aligned16(y) || (idx_out && !nm_aligned16(idx_out))) return NM_ERR_ALIGNMENT;
    if (dtype != NM_F32 && dtype != NM_BF16 && dtype != NM_F16) return NM_ERR_UNSUPPORTED;
    return nm_launch_pwl_apply(ctx, slot, x, y, count, dtype, idx_out, (cudaStream_t)stream);
}

nm_status nm_linear_pwl(nm_ctx* ctx, const nm_linear_desc* d, void* stream)
{
    if (!ctx || !d) return NM_ERR_INVALID_ARG;
    if (d->M < 0 || d->N < 0 || d->K < 0) return NM_ERR_SHAPE;
    if (d->slot != NM_SLOT_NONE) {
        nm_status s = need_table(ctx, d->slot);
        if (s != NM_OK) return s;
    }
    if (d->M == 0 || d->N == 0) return NM_OK;
    if (d->K == 0) return NM_ERR_SHAPE;
    if (!d->A || !d->W || !d->out) return NM_ERR_INVALID_ARG;
    if (d->in_dtype < NM_F32 || d->in_dtype > NM_I8 || d->out_dtype < NM_F32 || d->out_dtype > NM_I8)
        return NM_ERR_INVALID_ARG;
    if (d->lda < d->K || d->ldw < d->K || d->ldo < d->N || (d->residual && d->ldr < d->N)) return NM_ERR_SHAPE;
    const size_t es = nm_dtype_size(d->in_dtype), os = nm_dtype_size(d->out_dtype);
    if (!nm_aligned16(d->A) || !nm_aligned16(d->W) || !nm_aligned16(d->out) || !nm_aligned16(d->bias) ||
        !nm_aligned16(d->residual) || !nm_aligned16(d->w_scale) || !nm_aligned16(d->acc_dump) ||
        !nm_aligned16(d->idx_dump))
        return NM_ERR_ALIGNMENT;
    if ((d->lda * es) % 16 || (d->ldw * es) % 16 || (d->ldo * os) % 16 || (d->residual && (d->ldr * os) % 16))
        return NM_ERR_ALIGNMENT;
    if (d->in_dtype == NM_I8) {
        if (!d->w_scale) return NM_ERR_INVALID_ARG;
        if (d->out_dtype == NM_F16) return NM_ERR_UNSUPPORTED;
        if (d->out_dtype == NM_I8 && d->residual) return NM_ERR_UNSUPPORTED;
    } else {
        if (d->out_dtype != d->in_dtype) return NM_ERR_UNSUPPORTED;
        if (d->acc_dump) return NM_ERR_UNSUPPORTED;
    }
    cudaStream_t st = (cudaStream_t)stream;
    if (d->algo == 1) return nm_launch_linear_simt(ctx, d, st);
    const bool tc = nm_linear_tc_supported(d);
    if (d->algo == 2 || d->algo == 3) return tc ? nm_launch_linear_tc(ctx, d, st) : NM_ERR_UNSUPPORTED;
    // tiny problems do not fill a 128-row tensor-core tile; the CUDA-core kernel takes them
    if (tc && d->M >= 64 && d->N >= 64) return nm_launch_linear_tc(ctx, d, st);
    return nm_launch_linear_simt(ctx, d, st);
}

// out_q != nullptr asks for the output as int8 codes in out_q instead of d->out; *fused tells whether the
// kernel chosen could do that (the caller quantises d->out itself otherwise).
static nm_status attention_dispatch(nm_ctx* ctx, const nm_attn_desc* d, void* stream, int8_t* out_q,
                                    float q_inv_scale, bool* fused);

nm_status nm_attention_pwl(nm_ctx* ctx, const nm_attn_desc* d, void* stream)
{
    return attention_dispatch(ctx, d, stream, nullptr, 0.f, nullptr);
}

static nm_status attention_dispatch(nm_ctx* ctx, const nm_attn_desc* d, void* stream, int8_t* out_q,
                                    float q_inv_scale, bool* fused)
{
    if (fused) *fused = false;
    if (!ctx || !d) return NM_ERR_INVALID_ARG;
    if (d->B < 0 || d->L < 0 || d->heads < 0 || d->d < 0) return NM_ERR_SHAPE;
    nm_status s = need_table(ctx, d->exp_slot);
    if (s != NM_OK) return s;
    s = need_table(ctx, d->recip_slot);
    if (s != NM_OK) return s;
    if (d->B == 0 || d->L == 0 || d->heads == 0 || d->d == 0) return NM_OK;
    if (!d->Q || !d->K || !d->V || !d->out) return NM_ERR_INVALID_ARG;
    if (d->dtype != NM_F32 && d->dtype != NM_BF16 && d->dtype != NM_F16) return NM_ERR_UNSUPPORTED;
    if (!nm_aligned16(d->Q) || !nm_aligned16(d->K) || !nm_aligned16(d->V) || !nm_aligned16(d->out))
        return NM_ERR_ALIGNMENT;
    if (d->stride_t < (int64_t)d->heads * d->d || d->stride_b < (int64_t)d->L * d->stride_t) return NM_ERR_SHAPE;
    // the tensor-core kernels take the row maximum of the raw products and scale it afterwards, which
    // equals the maximum of the scaled scores only for a positive scale
    if (!(d->scale > 0.0f) || !isfinite(d->scale)) return NM_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (d->algo == 1) return nm_launch_attention_simt(ctx, d, st);
    // tensor-core kernels: the streaming one (several CTAs per SM, any L that is a multiple of 128) is the
    // default; algo 3 selects the one that keeps the whole score block in tensor memory (L <= 512)
    if (d->algo == 3) return nm_attention_tc_supported(d) ? nm_launch_attention_tc(ctx, d, st) : NM_ERR_UNSUPPORTED;
    if (d->algo == 0 && ctx->attn_resident && nm_attention_tc_supported(d)) {
        const nm_status s = nm_launch_attention_tc(ctx, d, st);
        if (s != NM_ERR_UNSUPPORTED) return s;
    }
    const bool tc = nm_attention_stream_supported(d);
    if (d->algo == 2) return tc ? nm_launch_attention_stream(ctx, d, st) : NM_ERR_UNSUPPORTED;
    if (tc) {
        const nm_status s = nm_launch_attention_stream(ctx, d, st, out_q, q_inv_scale);
        if (s != NM_ERR_UNSUPPORTED) {   // else: an exp table too large for shared memory
            if (fused && out_q && s == NM_OK) *fused = true;
            return s;
        }
    }
    return nm_launch_attention_simt(ctx, d, st);
}

nm_status nm_attention_pwl_i8(nm_ctx* ctx, const nm_attn_i8_desc* d, void* stream)
{
    if (!ctx || !d) return NM_ERR_INVALID_ARG;
    if (d->B < 0 || d->L < 0 || d->heads < 0 || d->d < 0) return NM_ERR_SHAPE;
    nm_status s = need_table(ctx, d->exp_slot);
    if (s != NM_OK) return s;
    s = need_table(ctx, d->recip_slot);
    if (s != NM_OK) return s;
    if (d->B == 0 || d->L == 0 || d->heads == 0 || d->d == 0) return NM_OK;
    if (!d->Q || !d->K || !d->V || !d->out) return NM_ERR_INVALID_ARG;
    if (d->out_dtype != NM_BF16 && d->out_dtype != NM_F32) return NM_ERR_UNSUPPORTED;
    if (!(d->scale > 0.0f) || !isfinite(d->scale) || !(d->s_q > 0.0f) || !(d->s_k > 0.0f) || !(d->s_v > 0.0f))
        return NM_ERR_INVALID_ARG;
    if (!nm_aligned16(d->Q) || !nm_aligned16(d->K) || !nm_aligned16(d->V) || !nm_aligned16(d->out) ||
        !nm_aligned16(d->acc_dump) || !nm_aligned16(d->p_dump) || !nm_aligned16(d->oacc_dump))
        return NM_ERR_ALIGNMENT;
    if (d->stride_t % 16 != 0 || d->stride_b % 16 != 0) return NM_ERR_ALIGNMENT;
    if (d->stride_t < (int64_t)d->heads * d->d || d->stride_b < (int64_t)d->L * d->stride_t) return NM_ERR_SHAPE;
    if (d->d != 64 || d->L % 128 != 0) return NM_ERR_UNSUPPORTED;
    // the replicated exp table must fit beside the tiles
    if ((size_t)(ctx->h_tables[d->exp_slot].n + 1) * 16 * sizeof(float2) > 16 * 1024) return NM_ERR_UNSUPPORTED;
    return nm_launch_attention_i8(ctx, d, (cudaStream_t)stream);
}

// q != nullptr: the kernel also writes the int8 codes of its (rounded) output, scale 1/q_inv_scale
static nm_status layernorm_checked(nm_ctx* ctx, const void* x, const float* gamma, const float* beta, void* y,
                                   int64_t rows, int32_t H, float eps, int32_t rsqrt_slot, nm_dtype dtype, void* stream,
                                   int8_t* q, float q_inv_scale)
{
    if (!ctx) return NM_ERR_INVALID_ARG;
    if (rows < 0 || H < 0) return NM_ERR_SHAPE;
    nm_status s = need_table(ctx, rsqrt_slot);
    if (s != NM_OK) return s;
    if (rows == 0 || H == 0) return NM_OK;
    if (!x || !y || !gamma || !beta) return NM_ERR_INVALID_ARG;
    if (H % 8 != 0) return NM_ERR_SHAPE;
    if (!nm_aligned16(x) || !nm_aligned16(y) || !nm_aligned16(gamma) || !nm_aligned16(beta)) return NM_ERR_ALIGNMENT;
    return nm_launch_layernorm(ctx, x, gamma, beta, y, rows, H, eps, rsqrt_slot, NM_SLOT_NONE, dtype, (cudaStream_t)stream,
                               q, q_inv_scale);
}

nm_status nm_layernorm_pwl(nm_ctx* ctx, const void* x, const float* gamma, const float* beta, void* y,
                           int64_t rows, int32_t H, float eps, int32_t rsqrt_slot, nm_dtype dtype, void* stream)
{
    return layernorm_checked(ctx, x, gamma, beta, y, rows, H, eps, rsqrt_slot, dtype, stream, nullptr, 0.f);
}

nm_status nm_layernorm_pwl_sqrt_recip(nm_ctx* ctx, const void* x, const float* gamma, const float* beta, void* y,
                                      int64_t rows, int32_t H, float eps, int32_t sqrt_slot, int32_t recip_slot,
                                      nm_dtype dtype, void* stream)
{
    if (!ctx) return NM_ERR_INVALID_ARG;
    if (rows < 0 || H < 0) return NM_ERR_SHAPE;
    nm_status s = need_table(ctx, sqrt_slot);
    if (s != NM_OK) return s;
    s = need_table(ctx, recip_slot);
    if (s != NM_OK) return s;
    if (rows == 0 || H == 0) return NM_OK;
    if (!x || !y || !gamma || !beta) return NM_ERR_INVALID_ARG;
    if (H % 8 != 0) return NM_ERR_SHAPE;
    if (!nm_aligned16(x) || !nm_aligned16(y) || !nm_aligned16(gamma) || !nm_aligned16(beta)) return NM_ERR_ALIGNMENT;
    return nm_launch_layernorm(ctx, x, gamma, beta, y, rows, H, eps, sqrt_slot, recip_slot, dtype, (cudaStream_t)stream);
}

nm_status nm_selftest_bounded_wait(nm_ctx* ctx, int64_t limit_cycles, void* stream)
{
    if (!ctx) return NM_ERR_INVALID_ARG;
    if (limit_cycles < 1 || limit_cycles > 4000000000LL) return NM_ERR_SHAPE;
    return nm_launch_wait_selftest(ctx, (long long)limit_cycles, (cudaStream_t)stream);
}

nm_status nm_quantize_i8(nm_ctx* ctx, const void* x, nm_dtype dtype, int64_t count, float inv_scale, int8_t* q,
                         void* stream)
{
    if (!ctx) return NM_ERR_INVALID_ARG;
    if (count < 0) return NM_ERR_SHAPE;
    if (count == 0) return NM_OK;
    if (!x || !q) return NM_ERR_INVALID_ARG;
    if (!nm_aligned16(x) || !nm_aligned16(q)) return NM_ERR_ALIGNMENT;
    return nm_launch_quantize(ctx, x, dtype, count, inv_scale, q, (cudaStream_t)stream);
}

// ---------------------------------------------------------------- encoder layer

static size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

struct EncLayout {
    size_t qkv, attn, z, x1, g, q8a, q8b, pingpong, total;
};

static bool enc_layout(const nm_encoder_cfg* c, EncLayout* lo)
{
    if (!c || c->B < 1 || c->L < 1 || c->H < 1 || c->heads < 1 || c->F < 1) return false;
    if (c->H % c->heads) return false;
    const size_t T = (size_t)c->B * c->L;
    const size_t as = c->dtype == NM_F32 ? 4 : 2;  // activation element size (bf16 for the int8 path)
    size_t o = 0;
    lo->qkv = o; o += align256(T * 3 * c->H * as);
    lo->attn = o; o += align256(T * c->H * as);
    lo->z = o; o += align256(T * c->H * as);
    lo->x1 = o; o += align256(T * c->H * as);
    lo->g = o; o += align256(T * c->F * as);
    lo->q8a = o; o += c->dtype == NM_I8 ? align256(T * (size_t)(c->H > c->F ? c->H : c->F)) : 0;
    lo->q8b = o; o += 0;
    lo->pingpong = o; o += align256(T * c->H * as);
    lo->total = o;
    return true;
}

size_t nm_encoder_workspace_bytes(const nm_encoder_cfg* cfg)
{
    EncLayout lo;
    if (!enc_layout(cfg, &lo)) return 0;
    return lo.total;
}

// The int8 layer quantises three activations (its input, the attention output, LN1's output).  The
// producing kernels write those int8 codes themselves where they can (LayerNorm and the streaming
// attention kernel), so no separate pass re-reads the activation.  Within a stack the previous layer's
// LN2 has already left the codes of this layer's input in the workspace (`in_codes_ready`), and this
// layer's LN2 leaves those of the next (`next_a_x` > 0: the next layer's input scale).
static nm_status encoder_layer_impl(nm_ctx* ctx, const nm_encoder_weights* w, const nm_encoder_cfg* c, const void* x,
                                    void* y, void* workspace, size_t ws_bytes, void* stream, bool in_codes_ready,
                                    float next_a_x);

nm_status nm_encoder_layer(nm_ctx* ctx, const nm_encoder_weights* w, const nm_encoder_cfg* c, const void* x, void* y,
                           void* workspace, size_t ws_bytes, void* stream)
{
    return encoder_layer_impl(ctx, w, c, x, y, workspace, ws_bytes, stream, false, 0.f);
}

static nm_status encoder_layer_impl(nm_ctx* ctx, const nm_encoder_weights* w, const nm_encoder_cfg* c, const void* x,
                                    void* y, void* workspace, size_t ws_bytes, void* stream, bool in_codes_ready,
                                    float next_a_x)
{
    if (!ctx || !w || !c || !x || !y) return NM_ERR_INVALID_ARG;
    EncLayout lo;
    if (!enc_layout(c, &lo)) return NM_ERR_SHAPE;
    if (!workspace || ws_bytes < lo.total) return NM_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255u) != 0) return NM_ERR_ALIGNMENT;
    if (x == y) return NM_ERR_INVALID_ARG;
    if (c->dtype != NM_F32 && c->dtype != NM_BF16 && c->dtype != NM_I8) return NM_ERR_UNSUPPORTED;
    const nm_dtype act = c->dtype == NM_F32 ? NM_F32 : NM_BF16;
    const bool i8 = c->dtype == NM_I8;
    const int64_t T = (int64_t)c->B * c->L;
    const int H = c->H, F = c->F, d = H / c->heads;
    uint8_t* ws = (uint8_t*)workspace;
    void* qkv = ws + lo.qkv;
    void* attn = ws + lo.attn;
    void* z = ws + lo.z;
    void* x1 = ws + lo.x1;
    void* g = ws + lo.g;
    int8_t* q8 = (int8_t*)(ws + lo.q8a);
    nm_status s;

    auto linear = [&](const void* A, int64_t K, const void* W, int64_t N, const float* bias, const void* res,
                      int slot, void* out, nm_dtype out_dt, float a_scale, const float* w_scale,
                      float inv_out_scale) -> nm_status {
        nm_linear_desc ld;
        memset(&ld, 0, sizeof(ld));
        ld.M = T; ld.N = N; ld.K = K;
        ld.in_dtype = i8 ? NM_I8 : act;
        ld.out_dtype = out_dt;
        ld.A = A; ld.lda = K; ld.W = W; ld.ldw = K;
        ld.bias = bias; ld.residual = res; ld.ldr = N;
        ld.slot = slot; ld.out = out; ld.ldo = N;
        ld.a_scale = a_scale; ld.w_scale = w_scale; ld.inv_out_scale = inv_out_scale;
        ld.algo = c->algo;
        return nm_linear_pwl(ctx, &ld, stream);
    };

    // qkv = x Wqkv^T + bqkv
    const void* a_in = x;
    if (i8) {
        if (!in_codes_ready) {
            s = nm_quantize_i8(ctx, x, act, T * H, 1.0f / w->a_x, q8, stream);
            if (s != NM_OK) return s;
        }
        a_in = q8;
    }
    s = linear(a_in, H, w->Wqkv, 3 * H, w->bqkv, nullptr, NM_SLOT_NONE, qkv, act, w->a_x, w->s_wqkv, 0.f);
    if (s != NM_OK) return s;

    // a = attention(qkv)
    nm_attn_desc ad;
    memset(&ad, 0, sizeof(ad));
    ad.B = c->B; ad.L = c->L; ad.heads = c->heads; ad.d = d; ad.dtype = act;
    const size_t as = nm_dtype_size(act);
    ad.Q = qkv; ad.K = (uint8_t*)qkv + (size_t)H * as; ad.V = (uint8_t*)qkv + (size_t)2 * H * as;
    ad.stride_b = (int64_t)c->L * 3 * H; ad.stride_t = 3 * H;
    ad.scale = 1.0f / sqrtf((float)d);
    ad.exp_slot = c->exp_slot; ad.recip_slot = c->recip_slot; ad.out = attn; ad.algo = c->algo;
    bool attn_codes = false;
    s = attention_dispatch(ctx, &ad, stream, i8 ? q8 : nullptr, i8 ? 1.0f / w->a_attn : 0.f, &attn_codes);
    if (s != NM_OK) return s;

    // z = x + a Wo^T + bo ; x1 = LN1(z)
    a_in = attn;
    if (i8) {
        if (!attn_codes) {
            s = nm_quantize_i8(ctx, attn, act, T * H, 1.0f / w->a_attn, q8, stream);
            if (s != NM_OK) return s;
        }
        a_in = q8;
    }
    s = linear(a_in, H, w->Wo, H, w->bo, x, NM_SLOT_NONE, z, act, w->a_attn, w->s_wo, 0.f);
    if (s != NM_OK) return s;
    s = layernorm_checked(ctx, z, w->g1, w->be1, x1, T, H, c->eps, c->rsqrt_slot, act, stream, i8 ? q8 : nullptr,
                          i8 ? 1.0f / w->a_x1 : 0.f);
    if (s != NM_OK) return s;

    // g = PWLgelu(x1 W1^T + b1)   (int8 path: requantised in the epilogue with the scale of g)
    a_in = i8 ? (const void*)q8 : (const void*)x1;
    if (i8) s = linear(a_in, H, w->W1, F, w->b1, nullptr, c->gelu_slot, g, NM_I8, w->a_x1, w->s_w1, 1.0f / w->a_g);
    else s = linear(a_in, H, w->W1, F, w->b1, nullptr, c->gelu_slot, g, act, 0.f, nullptr, 0.f);
    if (s != NM_OK) return s;

    // y = LN2(x1 + g W2^T + b2)
    s = linear(g, F, w->W2, H, w->b2, x1, NM_SLOT_NONE, z, act, w->a_g, w->s_w2, 0.f);
    if (s != NM_OK) return s;
    const bool chain = i8 && next_a_x > 0.f;
    return layernorm_checked(ctx, z, w->g2, w->be2, y, T, H, c->eps, c->rsqrt_slot, act, stream, chain ? q8 : nullptr,
                             chain ? 1.0f / next_a_x : 0.f);
}

nm_status nm_encoder_stack(nm_ctx* ctx, const nm_encoder_weights* layers, int32_t n_layers, const nm_encoder_cfg* c,
                           const void* x, void* y, void* workspace, size_t ws_bytes, void* stream)
{
    if (!ctx || !layers || !c || !x || !y) return NM_ERR_INVALID_ARG;
    if (n_layers < 1) return NM_ERR_SHAPE;
    EncLayout lo;
    if (!enc_layout(c, &lo)) return NM_ERR_SHAPE;
    if (!workspace || ws_bytes < lo.total) return NM_ERR_WORKSPACE;
    // layer outputs alternate between y and a workspace buffer so that the last one lands in y
    void* pp = (uint8_t*)workspace + lo.pingpong;
    const void* in = x;
    bool codes_ready = false;
    for (int l = 0; l < n_layers; ++l) {
        const bool to_y = ((n_layers - 1 - l) % 2) == 0;
        void* out = to_y ? y : pp;
        // int8: LN2 of layer l leaves the codes of layer l+1's input in the workspace
        const float next_a_x = (c->dtype == NM_I8 && l + 1 < n_layers) ? layers[l + 1].a_x : 0.f;
        nm_status s = encoder_layer_impl(ctx, &layers[l], c, in, out, workspace, ws_bytes, stream, codes_ready, next_a_x);
        codes_ready = next_a_x > 0.f;
        if (s != NM_OK) return s;
        in = out;
    }
    return NM_OK;
}

nm_status nm_encoder_stack_host_async(nm_ctx* ctx, const nm_encoder_weights* layers, int32_t n_layers,
                                      const nm_encoder_cfg* c, const void* x_host, void* y_host, void* x_dev,
                                      void* y_dev, void* workspace, size_t ws_bytes, void* stream)
{
    if (!ctx || !c || !x_host || !y_host || !x_dev || !y_dev) return NM_ERR_INVALID_ARG;
    if (c->B < 1 || c->L < 1 || c->H < 1) return NM_ERR_SHAPE;
    const size_t bytes = (size_t)c->B * c->L * c->H * (c->dtype == NM_F32 ? 4 : 2);
    cudaStream_t st = (cudaStream_t)stream;
    NM_CUDA_TRY(cudaMemcpyAsync(x_dev, x_host, bytes, cudaMemcpyHostToDevice, st));
    nm_status s = nm_encoder_stack(ctx, layers, n_layers, c, x_dev, y_dev, workspace, ws_bytes, stream);
    if (s != NM_OK) return s;
    NM_CUDA_TRY(cudaMemcpyAsync(y_host, y_dev, bytes, cudaMemcpyDeviceToHost, st));
    return NM_OK;
}

nm_status nm_encoder_stack_host(nm_ctx* ctx, const nm_encoder_weights* layers, int32_t n_layers,
                                const nm_encoder_cfg* c, const void* x_host, void* y_host, void* x_dev, void* y_dev,
                                void* workspace, size_t ws_bytes, void* stream)
{
    nm_status s = nm_encoder_stack_host_async(ctx, layers, n_layers, c, x_host, y_host, x_dev, y_dev, workspace,
                                              ws_bytes, stream);
    if (s != NM_OK) return s;
    NM_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    return NM_OK;
}

}  // extern "C"

// ---------------------------------------------------------------- encoder layer without a caller workspace

extern "C" nm_status nm_encoder_layer_static(nm_ctx* ctx, const nm_encoder_weights* w, const nm_encoder_cfg* cfg,
                                             const void* x, void* y, void* stream)
{
    if (!ctx || !w || !cfg || !x || !y) return NM_ERR_INVALID_ARG;
    const size_t need = nm_encoder_workspace_bytes(cfg);
    if (need == 0) return NM_ERR_SHAPE;
    if (need > (size_t)NM_STATIC_WS_BYTES) return NM_ERR_WORKSPACE;  // larger layers must bring their own workspace
    if (!ctx->static_ws) return NM_ERR_CUDA;   // the array's address could not be resolved when the context was made
    // per-launch event records (profiling) would create CUDA events: keep them off in this call
    const int prof = ctx->profiling;
    ctx->profiling = 0;
    const nm_status s = nm_encoder_layer(ctx, w, cfg, x, y, ctx->static_ws, (size_t)NM_STATIC_WS_BYTES, stream);
    ctx->profiling = prof;
    return s;
}
