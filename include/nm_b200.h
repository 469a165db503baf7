/*
 * nm_b200.h -- C ABI of the B200-native NeuralMatrix forward pass.
 *
 * NeuralMatrix (arXiv 2305.14405) runs a whole DNN as linear matrix operations:
 * linear operators become GEMMs (Section 3.1) and every nonlinear operator is
 * replaced by a continuous piecewise-linear (PWL) table evaluated as
 * y = k[s]*x + b[s], s being the segment x falls in (Section 3.2, Section
 * 3.2.1, Algorithm 3 line 1).  This library is that forward pass as hand-written
 * sm_100a kernels.
 *
 * Conventions for every call
 *  - Returns nm_status; never aborts, never traps.  nm_status_string() names a code.
 *  - "device pointer" = caller-owned CUDA device memory on the context's device;
 *    "host pointer" = ordinary host memory.  The library never frees or keeps a
 *    caller pointer after the call returns, except where stated.
 *  - Matrices are row-major with an explicit leading dimension in ELEMENTS.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *    stream).  Work is enqueued and the call returns without waiting unless
 *    stated otherwise.
 *  - Per-call scratch comes from the caller's workspace (nm_*_workspace_bytes).
 *    The library allocates device memory only in nm_ctx_create; while per-kernel timing
 *    (nm_ctx_profile_enable) is on, launches also create CUDA events the first time a record
 *    slot is used.
 *  - Device-side failures (a bounded wait that expired) are written to a status
 *    word in the context; read it with nm_ctx_poll_status.
 *  - bias, gamma, beta, scales are fp32 for every activation dtype.
 */
#ifndef NM_B200_H
#define NM_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    NM_OK = 0,
    NM_ERR_INVALID_ARG = 1, /* null pointer, bad enum, bad slot, bad count        */
    NM_ERR_SHAPE = 2,       /* a size the call cannot take (zero is fine: no-op)  */
    NM_ERR_ALIGNMENT = 3,   /* pointer or leading dimension not 16-byte aligned   */
    NM_ERR_NO_TABLE = 4,    /* the PWL slot named by the call was never loaded    */
    NM_ERR_UNSUPPORTED = 5, /* a dtype / shape combination with no kernel         */
    NM_ERR_CUDA = 6,        /* a CUDA runtime or driver call failed               */
    NM_ERR_TIMEOUT = 7,     /* a device-side bounded wait expired                 */
    NM_ERR_WORKSPACE = 8    /* workspace too small or null                        */
} nm_status;

typedef enum { NM_F32 = 0, NM_BF16 = 1, NM_F16 = 2, NM_I8 = 3 } nm_dtype;

/* PWL table slots.  A slot holds one table; kernels name the slot they use. */
enum {
    NM_SLOT_NONE = -1,
    NM_SLOT_GELU = 0,
    NM_SLOT_EXP = 1,
    NM_SLOT_RECIP = 2,
    NM_SLOT_RSQRT = 3,
    NM_SLOT_RELU = 4,
    NM_SLOT_USER0 = 5,
    NM_NUM_SLOTS = 16
};
#define NM_MAX_SEGMENTS 256

/* Functions nm_pwl_table_build knows. */
enum { NM_FUNC_GELU = 0, NM_FUNC_EXP = 1, NM_FUNC_RECIP = 2, NM_FUNC_RSQRT = 3, NM_FUNC_RELU = 4,
       NM_FUNC_SQRT = 5, NM_FUNC_IDENTITY = 6 };

typedef struct nm_ctx nm_ctx;

const char* nm_status_string(nm_status s);

/* Creates a context on CUDA device `device` (tables, status word, cached kernel
 * attributes).  *out is owned by the caller until nm_ctx_destroy. */
nm_status nm_ctx_create(nm_ctx** out, int device);
nm_status nm_ctx_destroy(nm_ctx* ctx);

/* Waits for `stream`, then copies the device status word to *device_status
 * (an nm_status; NM_OK if no kernel reported a failure) and clears it. */
nm_status nm_ctx_poll_status(nm_ctx* ctx, int* device_status, void* stream);

/* Host-only table construction (Section 3.2.1 "Post-Training Approximation" with
 * the parameters of Algorithm 3 line 1): n equal segments on [x_min, x_max],
 * segment i is the secant of `func` through its two breakpoints, so neighbouring
 * segments meet.  Computed in fp64, rounded once to fp32.
 * k_host, b_host: host arrays of n floats, written.  1 <= n <= NM_MAX_SEGMENTS. */
nm_status nm_pwl_table_build(int func, int n, float x_min, float x_max, float* k_host, float* b_host);

/* Host-only construction of an ELASTIC table (Section 3.2: Algorithm 1 without its training loop):
 * Algorithm 2 "Horizontal Size Optimization" walks [r_min, r_max] in primary segments of length dLx
 * and opens a new segment only where the primary slope differs from the slope remembered at the last
 * kept start point by more than dK_th; Algorithm 3 "Vertical Bias Correction" gives each segment its
 * secant k, b and, when bias_correct != 0, shifts b by dE = mean of func over the segment minus the mean
 * of the secant, if |dE| > e_th (the reading of the section's prose).
 * The result is returned on the PRIMARY grid: n_cells = (r_max - r_min)/dLx equal cells (at most
 * NM_MAX_SEGMENTS; the range must be a whole number of primary segments), every cell carrying the k, b of
 * the merged segment it belongs to, so the table loads with nm_pwl_table_load(slot, n_cells, r_min, r_max,
 * k, b) and the kernels evaluate it with the same one-FMA index as any other table.  *n_segments_out is
 * the number of distinct segments Algorithm 2 kept (the parameter count the paper reports on).
 * k_host, b_host: host arrays of NM_MAX_SEGMENTS floats. */
nm_status nm_pwl_table_build_elastic(int func, float r_min, float r_max, float dLx, float dK_th, int bias_correct,
                                     float e_th, int* n_cells_out, int* n_segments_out, float* k_host,
                                     float* b_host);

/* Copies a table into `slot` ("parameters k and b of each segment are pre-stored
 * ... and indexed by the segment number", Section 3.2).  The table has n equal
 * segments on [x_min, x_max]; k_host/b_host are host arrays of n floats and may
 * be freed on return.  The segment of an input x is
 *     s = clamp(floor(fma(x, inv_h, off)), 0, n-1),  one fp32 fused multiply-add,
 *     inv_h = (float)(n / (x_max - x_min)),  off = (float)(-x_min * n / (x_max - x_min)),
 * so inputs outside the range use the first / last segment's k and b
 * (Section 3.2.1); NaN selects segment 0.  Synchronous; must not be called while
 * kernels that read the slot are in flight. */
nm_status nm_pwl_table_load(nm_ctx* ctx, int slot, int n, float x_min, float x_max,
                            const float* k_host, const float* b_host);

/* Element-wise table evaluation y[i] = fma(k[s], x[i], b[s]) in fp32 (Section 3.2:
 * segment matrix S, then Y = X.K + B).  x, y: device pointers to `count` elements
 * of `dtype` (F32, BF16 or F16), 16-byte aligned; idx_out: device int32[count] or
 * NULL, receives the segment numbers. */
nm_status nm_pwl_apply(nm_ctx* ctx, int slot, const void* x, void* y, int64_t count, nm_dtype dtype,
                       int32_t* idx_out, void* stream);

/* Linear operator with PWL epilogue (Section 3.1 "linear operations ... can be
 * represented as matrix addition and multiplication"; Section 3.2 for the table):
 *     out = PWL_slot(A . W^T * scale + bias) + residual        (order: bias, table, residual)
 * A [M,K] and W [N,K] of in_dtype (both K-contiguous), device pointers.
 * bias: device float[N] or NULL.  residual: device [M,N] of out_dtype (leading
 * dimension ldr) or NULL.  slot: NM_SLOT_NONE for no table.
 * in_dtype F32/BF16/F16: out_dtype must equal in_dtype; fp32 accumulation.
 * in_dtype I8: int32 accumulation (exact), then in fp32
 *     x = fma((float)acc, a_scale * w_scale[j], bias[j]);  y = fma(k[s], x, b[s]);  y += residual;
 *   out_dtype BF16 / F32 stores y; out_dtype I8 stores clamp(rint(y * inv_out_scale), -127, 127)
 *   (ties to even; residual not allowed with I8 out).  w_scale: device float[N].
 *   acc_dump / idx_dump: device int32[M*N] (row-major, ld N) or NULL: the raw
 *   accumulators and the segment numbers, for bit-exact checks.
 * All pointers 16-byte aligned, lda/ldw/ldo/ldr multiples of 16 bytes.
 * algo: 0 = pick; 1 = force the plain SIMT kernel; 2 = force the tcgen05 kernel
 * (NM_ERR_UNSUPPORTED if the shape or dtype has none); 3 = tcgen05 with one CTA per
 * tile even where the two-CTA (cta_group::2) tile would be chosen. */
typedef struct {
    int64_t M, N, K;
    nm_dtype in_dtype;
    nm_dtype out_dtype;
    const void* A;
    int64_t lda;
    const void* W;
    int64_t ldw;
    const float* bias;
    const void* residual;
    int64_t ldr;
    int32_t slot;
    void* out;
    int64_t ldo;
    float a_scale;
    const float* w_scale;
    float inv_out_scale;
    int32_t* acc_dump;
    int32_t* idx_dump;
    int32_t algo;
    int32_t res_first;  /* nonzero: out = PWL(A.W^T*scale + bias + residual), the order a ResNet block needs */
} nm_linear_desc;

nm_status nm_linear_pwl(nm_ctx* ctx, const nm_linear_desc* desc, void* stream);

/* Multi-head attention with PWL softmax (attention is one of the linear operators
 * of Section 3.1; exp and 1/x are two of the functions approximated in Section
 * 3.2.2).  Per batch, head and query row i, over all L keys (no mask):
 *     s_j = scale * <q_i, k_j>;  m = max_j s_j;  e_j = PWL_exp(s_j - m);
 *     sigma = sum_j e_j;  r = PWL_recip(sigma);  o_i = sum_j (e_j * r) * v_j.
 * m is the maximum of the whole row (a PWL exponential is not multiplicative, so
 * a running-maximum rescaling would compute a different function).
 * Q, K, V: device pointers; element (batch b, token t, head g, channel c) is at
 * base[b*stride_b + t*stride_t + g*d + c], so the three may point into one packed
 * [B*L, 3*heads*d] projection.  out: device [B*L, heads*d], leading dimension
 * heads*d.  dtype F32, BF16 or F16 (fp32 arithmetic inside).  scale must be positive and finite
 * (NM_ERR_INVALID_ARG otherwise).
 * algo: 0 = pick; 1 = CUDA-core kernel; 2 = tensor-core kernel that streams K and V and computes
 * Q K^T twice (d = 64, L a multiple of 128); 3 = tensor-core kernel that keeps the whole score block
 * in tensor memory (d = 64, L in {128, 256, 384, 512}). */
typedef struct {
    int32_t B, L, heads, d;
    nm_dtype dtype;
    const void* Q;
    const void* K;
    const void* V;
    int64_t stride_b;
    int64_t stride_t;
    float scale;
    int32_t exp_slot;
    int32_t recip_slot;
    void* out;
    int32_t algo;
} nm_attn_desc;

nm_status nm_attention_pwl(nm_ctx* ctx, const nm_attn_desc* desc, void* stream);

/* INT8 attention: both matrix products of attention on int8 tensor cores with int32 accumulation (Section 5
 * evaluates whole INT8 networks; the paper fixes no scheme, this is the reading taken).  Q, K, V are int8
 * codes with per-tensor scales s_q, s_k, s_v; the probabilities are int8 codes of the fixed scale 1/127
 * (they lie in [0, 1]).  Per batch, head and query row i, with every integer exact and every fp32 step one
 * correctly rounded operation (so the result is defined bit for bit):
 *     acc_j = <q_i, k_j> (int32);  m = max_j acc_j;  sc = (s_q * s_k) * scale
 *     x_j = fma((float)acc_j, sc, -((float)m * sc));  e_j = PWL_exp(x_j)   [fp32 index and fma(k, x, b)]
 *     p_j = clamp(rint(e_j * 127), -127, 127);  sigma = (float)(sum_j p_j) * (1/127)   [integer row sum]
 *     o_c = sum_j p_j * v_jc (int32);  out_c = ((float)o_c * (s_v * (1/127))) * PWL_recip(sigma)
 * Element (batch b, token t, head g, channel c) of Q, K, V is at base[b*stride_b + t*stride_t + g*d + c]
 * (int8, strides in elements = bytes, multiples of 16), so the three may point into one packed [B*L, 3*heads*d]
 * tensor.  out: device [B*L, heads*d] of out_dtype (BF16 or F32).  d = 64, L a multiple of 128, scale > 0
 * (NM_ERR_UNSUPPORTED / NM_ERR_INVALID_ARG otherwise: this operator has the tensor-core kernel only).
 * acc_dump, p_dump: device int32 / int8 [B, heads, L, L] or NULL (the integer scores and the probability codes);
 * oacc_dump: device int32 [B*L, heads*d] or NULL (the integer P.V), for bit-exact checks. */
typedef struct {
    int32_t B, L, heads, d;
    const int8_t* Q;
    const int8_t* K;
    const int8_t* V;
    int64_t stride_b;
    int64_t stride_t;
    float s_q, s_k, s_v;
    float scale;
    int32_t exp_slot;
    int32_t recip_slot;
    void* out;
    nm_dtype out_dtype;
    int32_t* acc_dump;
    int8_t* p_dump;
    int32_t* oacc_dump;
} nm_attn_i8_desc;

nm_status nm_attention_pwl_i8(nm_ctx* ctx, const nm_attn_i8_desc* desc, void* stream);

/* LayerNorm with PWL reciprocal square root (Section 3.2.2 lists sqrt(x) and 1/x;
 * here fused into one rsqrt table):
 *     mu = mean(z);  v = mean((z - mu)^2);  r = PWL_rsqrt(v + eps);  y = (z - mu) * r * gamma + beta
 * x, y: device [rows, H] of dtype (F32/BF16/F16), contiguous rows; gamma, beta:
 * device float[H]. H must be a multiple of 8. */
nm_status nm_layernorm_pwl(nm_ctx* ctx, const void* x, const float* gamma, const float* beta, void* y,
                           int64_t rows, int32_t H, float eps, int32_t rsqrt_slot, nm_dtype dtype,
                           void* stream);

/* The same LayerNorm with the reciprocal square root taken as the two functions Section 3.2.2
 * itself lists, sqrt(x) and 1/x, one table each:
 *     r = PWL_recip(PWL_sqrt(v + eps))
 * sqrt_slot holds a table over the range of v + eps, recip_slot one over the range of its square
 * root (not the attention's 1/x table, whose range is that of the softmax row sums).  Arguments,
 * layout and errors as for nm_layernorm_pwl; NM_ERR_NO_TABLE if either slot is empty. */
nm_status nm_layernorm_pwl_sqrt_recip(nm_ctx* ctx, const void* x, const float* gamma, const float* beta, void* y,
                                      int64_t rows, int32_t H, float eps, int32_t sqrt_slot, int32_t recip_slot,
                                      nm_dtype dtype, void* stream);

/* Symmetric int8 quantisation of an activation tensor with a static scale:
 * q[i] = clamp(rint(x[i] * inv_scale), -127, 127), ties to even (the INT8
 * evaluation of Section 5).  x: device, `count` elements of dtype; q: device int8. */
nm_status nm_quantize_i8(nm_ctx* ctx, const void* x, nm_dtype dtype, int64_t count, float inv_scale,
                         int8_t* q, void* stream);

/* One post-LayerNorm transformer encoder layer computed entirely with GEMMs and
 * PWL tables (Section 5: BERT / RoBERTa):
 *     qkv = x Wqkv^T + bqkv;  a = attention(qkv);  x1 = LN1(x + a Wo^T + bo);
 *     g = PWL_gelu(x1 W1^T + b1);  y = LN2(x1 + g W2^T + b2)
 * Weights are device pointers: Wqkv [3H,H] (rows 0..H-1 give Q, then K, then V;
 * head g owns channels g*d..g*d+d-1), Wo [H,H], W1 [F,H], W2 [H,F] of the weight
 * dtype (cfg.dtype; int8 when cfg.dtype == NM_I8); biases and LayerNorm
 * parameters float.  For NM_I8: activations are bf16, the four weight GEMMs are
 * int8 with per-output-channel weight scales s_* (device float arrays) and static
 * per-tensor activation scales a_* (the scale of the tensor ENTERING that GEMM). */
typedef struct {
    const void* Wqkv; const float* bqkv;
    const void* Wo;   const float* bo;
    const float* g1;  const float* be1;
    const void* W1;   const float* b1;
    const void* W2;   const float* b2;
    const float* g2;  const float* be2;
    const float* s_wqkv; const float* s_wo; const float* s_w1; const float* s_w2;
    float a_x, a_attn, a_x1, a_g;
} nm_encoder_weights;

typedef struct {
    int32_t B, L, H, heads, F;
    nm_dtype dtype;           /* F32, BF16 (activations and weights) or I8 (bf16 activations) */
    float eps;
    int32_t gelu_slot, exp_slot, recip_slot, rsqrt_slot;
    int32_t algo;             /* as in nm_linear_desc, applied to every step */
} nm_encoder_cfg;

/* Bytes of device workspace nm_encoder_layer / nm_encoder_stack need (0 on bad cfg). */
size_t nm_encoder_workspace_bytes(const nm_encoder_cfg* cfg);

/* x, y: device [B*L, H] of the activation dtype; y may not alias x.
 * workspace: device, 256-byte aligned, at least nm_encoder_workspace_bytes. */
nm_status nm_encoder_layer(nm_ctx* ctx, const nm_encoder_weights* w, const nm_encoder_cfg* cfg,
                           const void* x, void* y, void* workspace, size_t ws_bytes, void* stream);

/* n_layers layers in sequence (`layers` is a HOST array of weight structs whose
 * members are device pointers); the output of one layer is the input of the next. */
nm_status nm_encoder_stack(nm_ctx* ctx, const nm_encoder_weights* layers, int32_t n_layers,
                           const nm_encoder_cfg* cfg, const void* x, void* y, void* workspace,
                           size_t ws_bytes, void* stream);

/* The same with HOST input and output: x_host is copied to the device, the stack
 * runs, the result is copied to y_host, and the call waits for the stream.
 * x_dev, y_dev: device staging buffers of B*L*H activation elements each. */
nm_status nm_encoder_stack_host(nm_ctx* ctx, const nm_encoder_weights* layers, int32_t n_layers,
                                const nm_encoder_cfg* cfg, const void* x_host, void* y_host,
                                void* x_dev, void* y_dev, void* workspace, size_t ws_bytes, void* stream);
/* The same without the final wait: the two copies and the kernels are only enqueued on `stream`; y_host
 * holds the result once the caller has synchronised that stream (or an event recorded after the call).
 * x_host and y_host should be page-locked so that the copies run asynchronously.  Calls on different
 * streams, each with its own x_dev, y_dev and workspace, may be in flight together (their copies then
 * overlap the other call's kernels); the tables of `ctx` must not be reloaded meanwhile. */
nm_status nm_encoder_stack_host_async(nm_ctx* ctx, const nm_encoder_weights* layers, int32_t n_layers,
                                      const nm_encoder_cfg* cfg, const void* x_host, void* y_host,
                                      void* x_dev, void* y_dev, void* workspace, size_t ws_bytes, void* stream);

/* 2-D convolution with PWL epilogue, NHWC (Section 3.1: convolution kernels are linear
 * operations whose matrix dimensions follow from width, height and channels; Section 3: ReLU
 * is already piecewise linear and is evaluated as a 2-segment table):
 *     out[n,oy,ox,co] = PWL( sum_{ky,kx,ci} x[n, oy*stride-pad+ky, ox*stride-pad+kx, ci] * w[co,ky,kx,ci]
 *                            + bias[co] ) + residual[n,oy,ox,co]          (zero padding)
 * or, with res_first != 0, PWL( ... + bias + residual ), the order of a ResNet block.
 * x [N,H,W,Cin], w [Cout,kh,kw,Cin], residual / out [N,Ho,Wo,Cout] with Ho = (H+2*pad-kh)/stride+1:
 * device pointers of dtype (F16 or BF16), 16-byte aligned; bias device float[Cout] or NULL
 * (BatchNorm is expected to be folded into w and bias by the caller).  Cout a multiple of 8;
 * Cin a multiple of 8, except that any Cin is taken by the gather path (kh*kw*Cin is then
 * padded to a multiple of 8).  It runs as a GEMM with M = N*Ho*Wo, K = kh*kw*Cin: 1x1 stride-1
 * convolutions read x directly, all others first gather their operand into `workspace`
 * (device, 256-byte aligned, at least nm_conv2d_workspace_bytes). */
typedef struct {
    int32_t N, H, W, Cin, Cout, kh, kw, stride, pad;
    nm_dtype dtype;
    const void* x;
    const void* w;
    const float* bias;
    const void* residual;
    int32_t slot;
    int32_t res_first;
    void* out;
    int32_t algo;
} nm_conv_desc;

size_t nm_conv2d_workspace_bytes(const nm_conv_desc* desc);
nm_status nm_conv2d_pwl(nm_ctx* ctx, const nm_conv_desc* desc, void* workspace, size_t ws_bytes, void* stream);

/* Max pooling, NHWC, window ks x ks, zero-size padding cells ignored (a maximum is itself
 * piecewise linear: max(a,b) = b + ReLU(a-b), Section 3), and global average pooling
 * [N,H,W,C] -> [N,C] (a linear operator, Section 3.1: multiplication by a constant 1/(H*W)
 * matrix).  The average runs as a GEMM on the tensor cores: one K-block per position, every
 * 64-channel block multiplied by the constant matrix (1/(H*W)) * identity, whose entry is rounded
 * to the storage type (relative 2^-11 for fp16, 2^-8 for bf16); images taller or wider than 256
 * positions are averaged on CUDA cores instead.  C a multiple of 8.  Calls on one context that
 * use different H*W or dtypes must not overlap on the GPU (they share the constant matrix). */
nm_status nm_maxpool2d(nm_ctx* ctx, const void* x, void* y, nm_dtype dtype, int32_t N, int32_t H, int32_t W,
                       int32_t C, int32_t ks, int32_t stride, int32_t pad, void* stream);
nm_status nm_avgpool_global(nm_ctx* ctx, const void* x, void* y, nm_dtype dtype, int32_t N, int32_t H, int32_t W,
                            int32_t C, void* stream);

/* The same max pooling with the maximum evaluated in that operator form (Section 3: every
 * operator is linear or a PWL table): over the window cells inside the image, in raster order,
 *     m = first cell;  m = m + PWL_relu(cell - m) for every further cell,
 * with the table in relu_slot (fp32 arithmetic).  With the 2-segment ReLU table the result equals
 * nm_maxpool2d's.  Arguments and errors as nm_maxpool2d; NM_ERR_NO_TABLE if the slot is empty. */
nm_status nm_maxpool2d_pwl(nm_ctx* ctx, const void* x, void* y, nm_dtype dtype, int32_t N, int32_t H, int32_t W,
                           int32_t C, int32_t ks, int32_t stride, int32_t pad, int32_t relu_slot, void* stream);

/* ResNet-50-shaped CNN computed entirely with GEMMs and PWL tables (Section 5 evaluates ResNet):
 * 7x7/2 convolution, 3x3/2 max-pool, 16 bottleneck blocks (1x1 -> 3x3 -> 1x1, widths 64/128/256/512
 * x4, the stride in the 3x3 convolution, 1x1 projection shortcut in the first block of a stage,
 * ReLU after every convolution and after the residual add), global average pool, fully connected.
 * convs: HOST array of NM_RESNET50_CONVS entries (device pointers inside) in network order:
 * conv1, then per block conv_a, conv_b, conv_c and, for the first block of a stage, the shortcut
 * projection.  x [batch,224,224,3] -> logits [batch, num_classes] of dtype (F16 or BF16);
 * num_classes a multiple of 8. */
#define NM_RESNET50_CONVS 53
typedef struct {
    const void* w;      /* [Cout, kh, kw, Cin] */
    const float* bias;  /* [Cout] */
} nm_conv_params;
typedef struct {
    int32_t batch;
    nm_dtype dtype;
    int32_t relu_slot;
    int32_t num_classes;
    int32_t algo;
    /* Variants of the network (Section 5 compares ResNet-50 "and its variant models" by depth and width): the
     * number of bottleneck blocks of the four stages and the width of the first stage (stage s has inner width
     * base_width << s and 4x that many output channels; the stem has base_width channels).  All zero = ResNet-50:
     * blocks {3, 4, 6, 3}, base_width 64.  blocks in 1..64; base_width a multiple of 8 in 8..256 (multiples of 64
     * take the implicit-GEMM convolutions throughout).  convs then holds 1 + sum over stages of (3 blocks + 1)
     * entries (nm_resnet_conv_count) and fc_w is [num_classes, 32 * base_width]. */
    int32_t blocks[4];
    int32_t base_width;
} nm_resnet50_cfg;
/* Entries of `convs` for a configuration (53 for ResNet-50); 0 if the configuration is not valid. */
int32_t nm_resnet_conv_count(const nm_resnet50_cfg* cfg);
size_t nm_resnet50_workspace_bytes(const nm_resnet50_cfg* cfg);
nm_status nm_resnet50_forward(nm_ctx* ctx, const nm_conv_params* convs, const void* fc_w, const float* fc_b,
                              const nm_resnet50_cfg* cfg, const void* x, void* logits, void* workspace,
                              size_t ws_bytes, void* stream);
/* The same with HOST input and output: x_host [batch,224,224,3] is copied to x_dev, the network
 * runs, logits_dev is copied to logits_host, and the call waits for the stream. */
nm_status nm_resnet50_forward_host(nm_ctx* ctx, const nm_conv_params* convs, const void* fc_w, const float* fc_b,
                                   const nm_resnet50_cfg* cfg, const void* x_host, void* logits_host, void* x_dev,
                                   void* logits_dev, void* workspace, size_t ws_bytes, void* stream);
/* The same without the final wait (see nm_encoder_stack_host_async). */
nm_status nm_resnet50_forward_host_async(nm_ctx* ctx, const nm_conv_params* convs, const void* fc_w,
                                         const float* fc_b, const nm_resnet50_cfg* cfg, const void* x_host,
                                         void* logits_host, void* x_dev, void* logits_dev, void* workspace,
                                         size_t ws_bytes, void* stream);

/* nm_encoder_layer for callers that cannot provide a workspace.  (The paper has no
 * counterpart to this call: it exists for the library's users, not for the method.)
 *
 * Some callers have no way to allocate device memory: code that runs inside a host framework
 * whose memory pool already owns the device's memory, a latency-critical serving loop in which
 * cudaMalloc and its implicit device-wide synchronisation are off-limits, or a plug-in that
 * receives only its input and output buffers.  For them the layer's scratch (the packed
 * projection, attention output, pre-LayerNorm sums, FFN hidden activations) lives in a fixed
 * array of NM_STATIC_WS_BYTES inside the library's device image; every GPU that loads the
 * library holds that array until the process exits.  The call itself performs no cudaMalloc,
 * cudaFree or other allocating call; per-launch profiling records are suspended for its
 * duration.  x, y, w, cfg, stream are exactly as in nm_encoder_layer.
 *
 * Limit: configurations with nm_encoder_workspace_bytes(cfg) > NM_STATIC_WS_BYTES return
 * NM_ERR_WORKSPACE (use nm_encoder_layer with your own workspace for those).
 * The array's device address is resolved once, by nm_ctx_create (cudaGetSymbolAddress with the
 * context's device current; that is also the moment the driver places the array on the device),
 * and kept in the context, so this call does no set-up of its own on any call, the first
 * included; NM_ERR_CUDA if that resolution failed.
 * All calls on a device share the one array and it keeps the previous call's
 * contents: nothing in it needs to start at zero (every buffer is fully written before it is
 * read), but two calls whose kernels overlap on the GPU (different streams, no ordering
 * between them) race on it. */
#define NM_STATIC_WS_BYTES (32u << 20)
nm_status nm_encoder_layer_static(nm_ctx* ctx, const nm_encoder_weights* w, const nm_encoder_cfg* cfg,
                                  const void* x, void* y, void* stream);

/* Diagnostic for the failure-detection path (no counterpart in the paper): launches a one-warp kernel
 * that waits on a barrier nothing ever arrives on.  Like every wait in the tensor-core kernels, the
 * wait is bounded: after limit_cycles SM clock cycles (1 .. 4e9) it gives up, writes NM_ERR_TIMEOUT to
 * the context's status word and the kernel returns normally, leaving the context usable.
 * nm_ctx_poll_status then reports NM_ERR_TIMEOUT. */
nm_status nm_selftest_bounded_wait(nm_ctx* ctx, int64_t limit_cycles, void* stream);

/* Number of kernels the library has launched through this context since creation
 * (or since the last call with reset != 0). */
int64_t nm_ctx_launch_count(nm_ctx* ctx, int reset);

/* Per-kernel timing for roofline reports.  While enabled, every kernel launch is
 * bracketed by a pair of CUDA events on the launching stream (a few microseconds of
 * overhead per launch, so throughput is measured with it off).  nm_ctx_profile_enable
 * clears earlier records; at most 8192 launches are recorded, later ones are dropped.
 * nm_ctx_profile_read waits for the recorded events and returns, for one kernel kind,
 * the number of launches, their summed duration in milliseconds and their summed
 * algorithmic work: floating-point or integer operations (2*M*N*K for a linear
 * operator, 4*B*heads*L*L*d for attention) for the tensor-core-bound kinds, bytes
 * read plus written (one pass each way) for the bandwidth-bound row kernels. */
enum { NM_KERNEL_PWL_APPLY = 0, NM_KERNEL_LAYERNORM = 1, NM_KERNEL_QUANTIZE = 2, NM_KERNEL_LINEAR_SIMT = 3,
       NM_KERNEL_LINEAR_TC = 4, NM_KERNEL_ATTENTION_SIMT = 5, NM_KERNEL_ATTENTION_TC = 6, NM_KERNEL_IM2COL = 7,
       NM_KERNEL_POOL = 8, NM_NUM_KERNEL_KINDS = 9 };
nm_status nm_ctx_profile_enable(nm_ctx* ctx, int on);
nm_status nm_ctx_profile_read(nm_ctx* ctx, int kind, int64_t* launches, double* total_ms, double* total_work);

#ifdef __cplusplus
}
#endif
#endif /* NM_B200_H */
