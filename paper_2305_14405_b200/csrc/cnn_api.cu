// C ABI of the CNN path: convolution as GEMM with PWL epilogue, pooling, and the
// ResNet-50-shaped network sequencing.  Arithmetic happens in the kernels launched from here.
#include <string.h>

#include "nm_common.cuh"

namespace {

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

// How a convolution reaches the tensor-core kernel.
enum ConvPath {
    CONV_DIRECT,    // 1x1, stride 1, no padding: the NHWC activation is the [M, Cin] GEMM operand as it stands
    CONV_IMPLICIT,  // Cin a multiple of 64: implicit GEMM, one 4-D TMA box of the activation per filter tap
    CONV_ROWTAP,    // Cin <= 8, kw <= 8 (an RGB first layer): implicit GEMM over a zero-padded 8-channel copy of the
                    // input, one K-block per filter row: 8 taps x 8 channels = 64 contiguous elements
    CONV_GATHER     // anything else: explicit gather (im2col) into the workspace, then the GEMM
};

struct ConvGeom {
    int Ho, Wo, K, Kpad;
    int64_t M;
    ConvPath path;
    bool pad_w;       // CONV_GATHER: weights need their rows padded to Kpad
    int Hp, Wp;       // CONV_ROWTAP: extent of the padded input copy
    size_t a_bytes, w_bytes;
};

bool conv_geom(const nm_conv_desc* d, ConvGeom* g)
{
    if (d->N < 1 || d->H < 1 || d->W < 1 || d->Cin < 1 || d->Cout < 1 || d->kh < 1 || d->kw < 1 || d->stride < 1 ||
        d->pad < 0)
        return false;
    if (d->H + 2 * d->pad < d->kh || d->W + 2 * d->pad < d->kw) return false;
    g->Ho = (d->H + 2 * d->pad - d->kh) / d->stride + 1;
    g->Wo = (d->W + 2 * d->pad - d->kw) / d->stride + 1;
    g->K = d->kh * d->kw * d->Cin;
    g->Kpad = (g->K + 7) & ~7;
    g->M = (int64_t)d->N * g->Ho * g->Wo;
    g->pad_w = false;
    g->Hp = g->Wp = 0;
    g->a_bytes = g->w_bytes = 0;
    if (d->kh == 1 && d->kw == 1 && d->stride == 1 && d->pad == 0 && d->Cin % 8 == 0) {
        g->path = CONV_DIRECT;
    } else if (d->Cin % 64 == 0 && d->algo != 1) {
        g->path = CONV_IMPLICIT;
    } else if (d->Cin <= 8 && d->kw <= 8 && d->algo != 1) {
        g->path = CONV_ROWTAP;
        // rows 0 .. (Ho-1)*s + kh - 1 and pixels 0 .. (Wo-1)*s + 7 of the padded copy are read
        g->Hp = (g->Ho - 1) * d->stride + d->kh;
        g->Wp = (g->Wo - 1) * d->stride + 8;
        if (g->Hp < d->H + d->pad) g->Hp = d->H + d->pad;   // (never read, but the copy kernel writes whole rows)
        g->a_bytes = align256((size_t)d->N * g->Hp * g->Wp * 8 * 2);
        g->w_bytes = align256((size_t)d->Cout * d->kh * 64 * 2);
    } else {
        g->path = CONV_GATHER;
        g->pad_w = g->Kpad != g->K;
        g->a_bytes = align256((size_t)g->M * g->Kpad * 2);
        g->w_bytes = g->pad_w ? align256((size_t)d->Cout * g->Kpad * 2) : 0;
    }
    return true;
}

// stage widths and block counts of the ResNet-50 topology
// depth per stage and first-stage width of a configuration (zeros: ResNet-50); false if not valid
struct ResnetShape {
    int blocks[4];
    int base;
};
bool resnet_shape(const nm_resnet50_cfg* c, ResnetShape* sh)
{
    const int def_blocks[4] = {3, 4, 6, 3};
    const bool all_zero = c->blocks[0] == 0 && c->blocks[1] == 0 && c->blocks[2] == 0 && c->blocks[3] == 0;
    for (int i = 0; i < 4; ++i) {
        sh->blocks[i] = all_zero ? def_blocks[i] : c->blocks[i];
        if (sh->blocks[i] < 1 || sh->blocks[i] > 64) return false;
    }
    sh->base = c->base_width == 0 ? 64 : c->base_width;
    return sh->base >= 8 && sh->base <= 256 && sh->base % 8 == 0;
}

}  // namespace

extern "C" {

size_t nm_conv2d_workspace_bytes(const nm_conv_desc* d)
{
    ConvGeom g;
    if (!d || !conv_geom(d, &g)) return 0;
    return g.a_bytes + g.w_bytes;
}

nm_status nm_conv2d_pwl(nm_ctx* ctx, const nm_conv_desc* d, void* workspace, size_t ws_bytes, void* stream)
{
    if (!ctx || !d) return NM_ERR_INVALID_ARG;
    ConvGeom g;
    if (!conv_geom(d, &g)) return NM_ERR_SHAPE;
    if (d->dtype != NM_F16 && d->dtype != NM_BF16) return NM_ERR_UNSUPPORTED;
    if (d->Cout % 8 != 0) return NM_ERR_SHAPE;
    if (!d->x || !d->w || !d->out) return NM_ERR_INVALID_ARG;
    if (!nm_aligned16(d->x) || !nm_aligned16(d->w) || !nm_aligned16(d->out) || !nm_aligned16(d->residual) ||
        !nm_aligned16(d->bias))
        return NM_ERR_ALIGNMENT;
    const size_t need = g.a_bytes + g.w_bytes;
    if (need > 0) {
        if (!workspace || ws_bytes < need) return NM_ERR_WORKSPACE;
        if (((uintptr_t)workspace & 255u) != 0) return NM_ERR_ALIGNMENT;
    }
    cudaStream_t st = (cudaStream_t)stream;
    if (g.path == CONV_IMPLICIT || g.path == CONV_ROWTAP) {
        NmConvTc c;
        memset(&c, 0, sizeof(c));
        c.dtype = d->dtype;
        c.N = d->N; c.Ho = g.Ho; c.Wo = g.Wo; c.Cout = d->Cout;
        c.bias = d->bias; c.residual = d->residual; c.slot = d->slot; c.res_first = d->res_first; c.out = d->out;
        c.algo = d->algo;
        c.flops = 2.0 * (double)g.M * d->Cout * g.K;
        if (g.path == CONV_IMPLICIT) {
            c.a_base = d->x;
            c.a_dim[0] = (uint64_t)d->Cin; c.a_dim[1] = (uint64_t)d->W; c.a_dim[2] = (uint64_t)d->H; c.a_dim[3] = (uint64_t)d->N;
            c.a_stride[0] = (uint64_t)d->Cin * 2; c.a_stride[1] = (uint64_t)d->W * d->Cin * 2;
            c.a_stride[2] = (uint64_t)d->H * d->W * d->Cin * 2;
            c.sw = c.sh = d->stride; c.pw = c.ph = d->pad;
            c.taps_y = d->kh; c.taps_x = d->kw; c.cblocks = d->Cin / 64;
            c.w = d->w; c.ldw = g.K; c.Ktot = g.K;
        } else {
            // the input with its border and five zero channels written out once (xp), the weights likewise (wp);
            // output pixel ox then reads the 64 contiguous elements of pixels ox*s .. ox*s + 7 of row oy*s + ky
            void* xp = workspace;
            void* wp = (uint8_t*)workspace + g.a_bytes;
            nm_status s = nm_launch_pad_input(ctx, d->x, xp, d->dtype, d->N, d->H, d->W, d->Cin, d->pad, g.Hp, g.Wp, st);
            if (s != NM_OK) return s;
            s = nm_launch_pad_weight(ctx, d->w, wp, d->dtype, d->Cout, d->kh, d->kw, d->Cin, st);
            if (s != NM_OK) return s;
            c.a_base = xp;
            c.a_dim[0] = 64; c.a_dim[1] = (uint64_t)g.Wo; c.a_dim[2] = (uint64_t)g.Hp; c.a_dim[3] = (uint64_t)d->N;
            c.a_stride[0] = (uint64_t)d->stride * 8 * 2;          // next output pixel: `stride` input pixels on
            c.a_stride[1] = (uint64_t)g.Wp * 8 * 2;
            c.a_stride[2] = (uint64_t)g.Hp * g.Wp * 8 * 2;
            c.sw = 1; c.sh = d->stride; c.pw = 0; c.ph = 0;
            c.taps_y = d->kh; c.taps_x = 1; c.cblocks = 1;
            c.w = wp; c.ldw = (int64_t)d->kh * 64; c.Ktot = (int64_t)d->kh * 64;
        }
        return nm_launch_conv_tc(ctx, &c, st);
    }
    const void* A = d->x;
    const void* Wm = d->w;
    int64_t Kg = g.K;
    if (g.path == CONV_GATHER) {
        void* a_buf = workspace;
        nm_status s = nm_launch_im2col(ctx, d->x, a_buf, d->dtype, d->N, d->H, d->W, d->Cin, d->kh, d->kw, d->stride,
                                       d->pad, g.Ho, g.Wo, g.Kpad, st);
        if (s != NM_OK) return s;
        A = a_buf;
        Kg = g.Kpad;
        if (g.pad_w) {
            void* w_buf = (uint8_t*)workspace + g.a_bytes;
            s = nm_launch_pad_rows(ctx, d->w, w_buf, d->dtype, d->Cout, g.K, g.Kpad, st);
            if (s != NM_OK) return s;
            Wm = w_buf;
        }
    }
    nm_linear_desc ld;
    memset(&ld, 0, sizeof(ld));
    ld.M = g.M; ld.N = d->Cout; ld.K = Kg;
    ld.in_dtype = d->dtype; ld.out_dtype = d->dtype;
    ld.A = A; ld.lda = Kg; ld.W = Wm; ld.ldw = Kg;
    ld.bias = d->bias; ld.residual = d->residual; ld.ldr = d->Cout;
    ld.slot = d->slot; ld.out = d->out; ld.ldo = d->Cout;
    ld.algo = d->algo; ld.res_first = d->res_first;
    return nm_linear_pwl(ctx, &ld, stream);
}

nm_status nm_maxpool2d(nm_ctx* ctx, const void* x, void* y, nm_dtype dtype, int32_t N, int32_t H, int32_t W, int32_t C,
                       int32_t ks, int32_t stride, int32_t pad, void* stream)
{
    if (!ctx || !x || !y) return NM_ERR_INVALID_ARG;
    if (dtype != NM_F16 && dtype != NM_BF16) return NM_ERR_UNSUPPORTED;
    if (N < 1 || H < 1 || W < 1 || C < 8 || C % 8 != 0 || ks < 1 || stride < 1 || pad < 0 || pad >= ks ||
        H + 2 * pad < ks || W + 2 * pad < ks)
        return NM_ERR_SHAPE;
    if (!nm_aligned16(x) || !nm_aligned16(y)) return NM_ERR_ALIGNMENT;
    const int Ho = (H + 2 * pad - ks) / stride + 1, Wo = (W + 2 * pad - ks) / stride + 1;
    return nm_launch_maxpool(ctx, x, y, dtype, N, H, W, C, ks, stride, pad, Ho, Wo, (cudaStream_t)stream);
}

nm_status nm_maxpool2d_pwl(nm_ctx* ctx, const void* x, void* y, nm_dtype dtype, int32_t N, int32_t H, int32_t W,
                           int32_t C, int32_t ks, int32_t stride, int32_t pad, int32_t relu_slot, void* stream)
{
    if (!ctx || !x || !y) return NM_ERR_INVALID_ARG;
    if (relu_slot < 0 || relu_slot >= NM_NUM_SLOTS) return NM_ERR_INVALID_ARG;
    if (!ctx->h_tables[relu_slot].loaded) return NM_ERR_NO_TABLE;
    if (dtype != NM_F16 && dtype != NM_BF16) return NM_ERR_UNSUPPORTED;
    if (N < 1 || H < 1 || W < 1 || C < 8 || C % 8 != 0 || ks < 1 || stride < 1 || pad < 0 || pad >= ks ||
        H + 2 * pad < ks || W + 2 * pad < ks)
        return NM_ERR_SHAPE;
    if (!nm_aligned16(x) || !nm_aligned16(y)) return NM_ERR_ALIGNMENT;
    const int Ho = (H + 2 * pad - ks) / stride + 1, Wo = (W + 2 * pad - ks) / stride + 1;
    return nm_launch_maxpool(ctx, x, y, dtype, N, H, W, C, ks, stride, pad, Ho, Wo, (cudaStream_t)stream, relu_slot);
}

nm_status nm_avgpool_global(nm_ctx* ctx, const void* x, void* y, nm_dtype dtype, int32_t N, int32_t H, int32_t W,
                            int32_t C, void* stream)
{
    if (!ctx || !x || !y) return NM_ERR_INVALID_ARG;
    if (dtype != NM_F16 && dtype != NM_BF16) return NM_ERR_UNSUPPORTED;
    if (N < 1 || H < 1 || W < 1 || C < 8 || C % 8 != 0) return NM_ERR_SHAPE;
    if (!nm_aligned16(x) || !nm_aligned16(y)) return NM_ERR_ALIGNMENT;
    cudaStream_t st = (cudaStream_t)stream;
    if (H > 256 || W > 256) return nm_launch_avgpool(ctx, x, y, dtype, N, H * W, C, st);   // beyond a TMA box: CUDA cores
    // As a GEMM on the tensor cores: out[n, c] = sum over the H*W positions p and the 64 channels c' of c's block of
    // x[n, p, c'] * D[c', c], D = (1/HW) * identity.  The implicit-GEMM kernel takes one K-block per position; column
    // tile t reads channel block t and multiplies by the one constant 64 x 64 matrix D kept in the context.
    if (ctx->pool_w_hw != H * W || ctx->pool_w_dtype != (int)dtype + 1) {
        nm_status s = nm_launch_fill_diag(ctx, ctx->d_pool_w, dtype, 1.0f / (float)(H * W), st);
        if (s != NM_OK) return s;
        ctx->pool_w_hw = H * W;
        ctx->pool_w_dtype = (int)dtype + 1;
    }
    NmConvTc c;
    memset(&c, 0, sizeof(c));
    c.dtype = dtype;
    c.a_base = x;
    c.a_dim[0] = (uint64_t)C; c.a_dim[1] = (uint64_t)W; c.a_dim[2] = (uint64_t)H; c.a_dim[3] = (uint64_t)N;
    c.a_stride[0] = (uint64_t)C * 2; c.a_stride[1] = (uint64_t)W * C * 2; c.a_stride[2] = (uint64_t)H * W * C * 2;
    c.sw = c.sh = 1; c.pw = c.ph = 0;
    c.taps_y = H; c.taps_x = W; c.cblocks = 1;
    c.w = ctx->d_pool_w; c.ldw = 64; c.Ktot = 64;
    c.N = N; c.Ho = 1; c.Wo = 1; c.Cout = C;
    c.slot = NM_SLOT_NONE; c.out = y;
    c.depthwise = 1;
    c.flops = 2.0 * (double)N * C * H * W;
    return nm_launch_conv_tc(ctx, &c, st);
}

// Workspace: four activation buffers of the largest activation (batch x 112 x 112 x base =
// batch x 56 x 56 x 4 base elements), one pooled vector, and the largest gather buffer (conv1).
static void resnet_layout(const nm_resnet50_cfg* c, const ResnetShape& sh, size_t* act, size_t* pooled, size_t* gather,
                          size_t* total)
{
    const size_t base = (size_t)sh.base;
    *act = align256((size_t)c->batch * 112 * 112 * base * 2);
    *pooled = align256((size_t)c->batch * 32 * base * 2);
    size_t g = align256((size_t)c->batch * 112 * 112 * 152 * 2) + align256(base * 152 * 2);  // conv1: K 147 -> 152
    const size_t g3 = align256((size_t)c->batch * 56 * 56 * 9 * base * 2);                   // stage-1 3x3
    if (g3 > g) g = g3;
    *gather = g;
    *total = 4 * *act + *pooled + *gather;
}

size_t nm_resnet50_workspace_bytes(const nm_resnet50_cfg* cfg)
{
    ResnetShape sh;
    if (!cfg || cfg->batch < 1 || !resnet_shape(cfg, &sh)) return 0;
    size_t act, pooled, gather, total;
    resnet_layout(cfg, sh, &act, &pooled, &gather, &total);
    return total;
}

int32_t nm_resnet_conv_count(const nm_resnet50_cfg* cfg)
{
    ResnetShape sh;
    if (!cfg || !resnet_shape(cfg, &sh)) return 0;
    int n = 1;
    for (int st = 0; st < 4; ++st) n += 3 * sh.blocks[st] + 1;
    return n;
}

nm_status nm_resnet50_forward(nm_ctx* ctx, const nm_conv_params* convs, const void* fc_w, const float* fc_b,
                              const nm_resnet50_cfg* cfg, const void* x, void* logits, void* workspace, size_t ws_bytes,
                              void* stream)
{
    if (!ctx || !convs || !fc_w || !cfg || !x || !logits) return NM_ERR_INVALID_ARG;
    if (cfg->batch < 1 || cfg->num_classes < 8 || cfg->num_classes % 8 != 0) return NM_ERR_SHAPE;
    if (cfg->dtype != NM_F16 && cfg->dtype != NM_BF16) return NM_ERR_UNSUPPORTED;
    ResnetShape sh;
    if (!resnet_shape(cfg, &sh)) return NM_ERR_SHAPE;
    const int base = sh.base, n_convs = nm_resnet_conv_count(cfg);
    size_t act, pooled, gather, total;
    resnet_layout(cfg, sh, &act, &pooled, &gather, &total);
    if (!workspace || ws_bytes < total) return NM_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255u) != 0) return NM_ERR_ALIGNMENT;
    uint8_t* ws = (uint8_t*)workspace;
    void* buf[4] = {ws, ws + act, ws + 2 * act, ws + 3 * act};
    void* pool_buf = ws + 4 * act;
    void* gather_buf = ws + 4 * act + pooled;
    const int Nb = cfg->batch;
    int ci = 0;  // index into convs

    auto conv = [&](const void* in, int H, int W, int Cin, int Cout, int k, int stride, int pad, const void* res,
                    int res_first, void* out) -> nm_status {
        nm_conv_desc d;
        memset(&d, 0, sizeof(d));
        d.N = Nb; d.H = H; d.W = W; d.Cin = Cin; d.Cout = Cout; d.kh = k; d.kw = k; d.stride = stride; d.pad = pad;
        d.dtype = cfg->dtype;
        d.x = in; d.w = convs[ci].w; d.bias = convs[ci].bias;
        d.residual = res; d.slot = cfg->relu_slot; d.res_first = res_first; d.out = out; d.algo = cfg->algo;
        ++ci;
        return nm_conv2d_pwl(ctx, &d, gather_buf, gather, stream);
    };

    // stem: 7x7/2 convolution + ReLU, 3x3/2 max-pool
    nm_status s = conv(x, 224, 224, 3, base, 7, 2, 3, nullptr, 0, buf[0]);
    if (s != NM_OK) return s;
    s = nm_maxpool2d(ctx, buf[0], buf[1], cfg->dtype, Nb, 112, 112, base, 3, 2, 1, stream);
    if (s != NM_OK) return s;
    int cur = 1;  // buffer holding the block input
    int H = 56, Cin = base;
    for (int st = 0; st < 4; ++st) {
        const int width = base << st, Cout = 4 * width;
        for (int b = 0; b < sh.blocks[st]; ++b) {
            const int stride = (b == 0 && st > 0) ? 2 : 1;
            const int Ho = H / stride;
            // the three free buffers
            int f[3], nf = 0;
            for (int i = 0; i < 4; ++i) if (i != cur) f[nf++] = i;
            void* t1 = buf[f[0]];
            void* t2 = buf[f[1]];
            void* sc = buf[f[2]];
            s = conv(buf[cur], H, H, Cin, width, 1, 1, 0, nullptr, 0, t1);          // 1x1 + ReLU
            if (s != NM_OK) return s;
            s = conv(t1, H, H, width, width, 3, stride, 1, nullptr, 0, t2);         // 3x3 (stride) + ReLU
            if (s != NM_OK) return s;
            // 1x1 + shortcut, ReLU after the add (res_first); conv_c precedes the projection in `convs`
            const nm_conv_params pc = convs[ci];
            const void* shortcut = buf[cur];
            if (b == 0) {
                ++ci;  // projection shortcut: its parameters follow conv_c
                const nm_conv_params pd = convs[ci];
                nm_conv_desc d;
                memset(&d, 0, sizeof(d));
                d.N = Nb; d.H = H; d.W = H; d.Cin = Cin; d.Cout = Cout; d.kh = 1; d.kw = 1; d.stride = stride; d.pad = 0;
                d.dtype = cfg->dtype; d.x = buf[cur]; d.w = pd.w; d.bias = pd.bias; d.slot = NM_SLOT_NONE; d.out = sc;
                d.algo = cfg->algo;
                s = nm_conv2d_pwl(ctx, &d, gather_buf, gather, stream);
                if (s != NM_OK) return s;
                shortcut = sc;
                --ci;
            }
            {
                nm_conv_desc d;
                memset(&d, 0, sizeof(d));
                d.N = Nb; d.H = Ho; d.W = Ho; d.Cin = width; d.Cout = Cout; d.kh = 1; d.kw = 1; d.stride = 1; d.pad = 0;
                d.dtype = cfg->dtype; d.x = t2; d.w = pc.w; d.bias = pc.bias; d.residual = shortcut;
                d.slot = cfg->relu_slot; d.res_first = 1; d.out = t1; d.algo = cfg->algo;
                s = nm_conv2d_pwl(ctx, &d, gather_buf, gather, stream);
                if (s != NM_OK) return s;
            }
            ci += (b == 0) ? 2 : 1;
            cur = f[0];  // t1 now holds the block output
            H = Ho;
            Cin = Cout;
        }
    }
    if (ci != n_convs) return NM_ERR_INVALID_ARG;
    const int feat = 32 * base;   // channels of the last stage
    s = nm_avgpool_global(ctx, buf[cur], pool_buf, cfg->dtype, Nb, 7, 7, feat, stream);
    if (s != NM_OK) return s;
    nm_linear_desc ld;
    memset(&ld, 0, sizeof(ld));
    ld.M = Nb; ld.N = cfg->num_classes; ld.K = feat;
    ld.in_dtype = cfg->dtype; ld.out_dtype = cfg->dtype;
    ld.A = pool_buf; ld.lda = feat; ld.W = fc_w; ld.ldw = feat; ld.bias = fc_b;
    ld.slot = NM_SLOT_NONE; ld.out = logits; ld.ldo = cfg->num_classes; ld.algo = cfg->algo;
    return nm_linear_pwl(ctx, &ld, stream);
}

nm_status nm_resnet50_forward_host_async(nm_ctx* ctx, const nm_conv_params* convs, const void* fc_w,
                                         const float* fc_b, const nm_resnet50_cfg* cfg, const void* x_host,
                                         void* logits_host, void* x_dev, void* logits_dev, void* workspace,
                                         size_t ws_bytes, void* stream)
{
    if (!ctx || !cfg || !x_host || !logits_host || !x_dev || !logits_dev) return NM_ERR_INVALID_ARG;
    if (cfg->batch < 1 || cfg->num_classes < 1) return NM_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t xb = (size_t)cfg->batch * 224 * 224 * 3 * 2, lb = (size_t)cfg->batch * cfg->num_classes * 2;
    NM_CUDA_TRY(cudaMemcpyAsync(x_dev, x_host, xb, cudaMemcpyHostToDevice, st));
    nm_status s = nm_resnet50_forward(ctx, convs, fc_w, fc_b, cfg, x_dev, logits_dev, workspace, ws_bytes, stream);
    if (s != NM_OK) return s;
    NM_CUDA_TRY(cudaMemcpyAsync(logits_host, logits_dev, lb, cudaMemcpyDeviceToHost, st));
    return NM_OK;
}

nm_status nm_resnet50_forward_host(nm_ctx* ctx, const nm_conv_params* convs, const void* fc_w, const float* fc_b,
                                   const nm_resnet50_cfg* cfg, const void* x_host, void* logits_host, void* x_dev,
                                   void* logits_dev, void* workspace, size_t ws_bytes, void* stream)
{
    nm_status s = nm_resnet50_forward_host_async(ctx, convs, fc_w, fc_b, cfg, x_host, logits_host, x_dev, logits_dev,
                                                 workspace, ws_bytes, stream);
    if (s != NM_OK) return s;
    NM_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    return NM_OK;
}

}  // extern "C"
