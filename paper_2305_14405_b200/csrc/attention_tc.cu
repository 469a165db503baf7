// Fused attention with PWL softmax on the 5th-generation tensor cores.
//
// Attention is one of the linear operators of Section 3.1; its softmax uses two of the
// functions Section 3.2.2 approximates, exp and 1/x, here as PWL tables.  Per query row:
//     s_j = scale*<q,k_j>;  m = max_j s_j;  e_j = PWL_exp(s_j - m);
//     sigma = sum_j e_j;    o = PWL_recip(sigma) * sum_j e_j v_j
// A PWL exponential is not multiplicative, so the row maximum must be the FINAL one:
// the whole score row block S = Q K^T (128 x L fp32) is kept in tensor memory, read once
// for the maximum and once more for the exponentials.  No running-maximum rescaling.
//
// One CTA per (batch, head, 128 query rows); head dimension 64; L in {128,256,384,512}.
//   warp 0        one lane: TMA loads of Q, K, V (128-byte swizzle), tcgen05.mma for
//                 S = Q K^T (K-major operands) and O += P V (V as an MN-major operand,
//                 straight from its [keys, d] layout), commits on mbarriers
//   warps 1..4*NH softmax warps, NH per tensor-memory lane quarter.  Warp group h owns the
//                 64-key chunks c with c % NH == h in both passes: tcgen05.ld of S, row
//                 maximum and row sum without shuffles (one thread owns a row of its
//                 chunks; the groups exchange through shared memory), PWL exp from a
//                 per-lane replicated table, P written to shared memory as bf16 in the
//                 swizzled K-major layout the MMA reads, PWL reciprocal, scaling, store.
// For L = 512 the S block fills all 512 tensor-memory columns; O then reuses columns
// 0..63, which are dead once the first 64 exponentials of every row are in P.
#include <string.h>

#include "nm_common.cuh"

namespace {

constexpr int BQ = 128;    // query rows per CTA
constexpr int HD = 64;     // head dimension
constexpr int ROWB = 128;  // bytes per tile row (64 x 16-bit)
constexpr int MAX_PBUF = 4;

struct AttnArgs {
    int B, L, heads;
    float scale;
    const NmTable* t_exp;
    const NmTable* t_rcp;
    void* out;
    int* status;
    int n_exp;
    int nbuf;    // P buffers
    int p_in_k;  // P buffers reuse the K tile region (L >= 256)
    uint32_t tmem_cols, o_col;
};

template <typename T> struct AttnT;
template <> struct AttnT<__nv_bfloat16> {
    static constexpr uint32_t fmt = 1;
    static __device__ __forceinline__ uint32_t pack(float a, float b)
    {
        __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
        return *reinterpret_cast<uint32_t*>(&h);
    }
};
template <> struct AttnT<__half> {
    static constexpr uint32_t fmt = 0;
    static __device__ __forceinline__ uint32_t pack(float a, float b)
    {
        __half2 h = __floats2half2_rn(a, b);
        return *reinterpret_cast<uint32_t*>(&h);
    }
};

__device__ __forceinline__ float max3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// 32 lanes x 16 consecutive 32-bit columns of tensor memory
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]),
                   "+r"(r[15]));
}

// NH: softmax warps per lane quarter.  CLAMP_HI: clamp the segment number from above; not
// needed when the exp table's range reaches 0 (its input, score minus row maximum, is never
// positive), the table copy in shared memory then carries one duplicated entry for input 0.
template <typename T, int NH, bool CLAMP_HI>
__global__ void __launch_bounds__(32 + 128 * NH)
attention_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const AttnArgs a)
{
    constexpr int NTHREADS = 32 + 128 * NH;
    constexpr int NSOFT = 128 * NH;
    constexpr uint32_t IDESC_QK = nm_idesc(1, AttnT<T>::fmt, 0, 0, BQ, 128);  // S chunk: 128 x 128
    constexpr uint32_t IDESC_PV = nm_idesc(1, AttnT<T>::fmt, 0, 1, BQ, HD);   // O: 128 x 64, V MN-major

    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_qk, bar_v, bar_s, bar_o, bar_drain;
    __shared__ uint64_t bar_p_full[MAX_PBUF], bar_p_empty[MAX_PBUF];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ float s_red[NH][BQ];  // row maximum / row sum exchange between the warp groups

    const int L = a.L;
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* q_s = base;                      // 128 x 128 B
    uint8_t* k_s = q_s + BQ * ROWB;           // L x 128 B
    uint8_t* v_s = k_s + (size_t)L * ROWB;    // L x 128 B
    uint8_t* extra = v_s + (size_t)L * ROWB;  // P buffers when they do not fit in K's region
    uint8_t* p_s = a.p_in_k ? k_s : extra;
    float2* rep = reinterpret_cast<float2*>(extra + (a.p_in_k ? 0 : (size_t)a.nbuf * BQ * ROWB));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int blocks_per_seq = L / BQ;
    const int qb = blockIdx.x % blocks_per_seq;
    const int g = (blockIdx.x / blocks_per_seq) % a.heads;
    const int b = blockIdx.x / (blocks_per_seq * a.heads);

    if (threadIdx.x == 0) {
        abort_flag = 0;
        nm_prefetch_tmap(&tmQ);
        nm_prefetch_tmap(&tmK);
        nm_prefetch_tmap(&tmV);
        nm_mbar_init(&bar_qk, 1);
        nm_mbar_init(&bar_v, 1);
        nm_mbar_init(&bar_s, 1);
        nm_mbar_init(&bar_o, 1);
        nm_mbar_init(&bar_drain, 1);
        for (int i = 0; i < MAX_PBUF; ++i) {
            nm_mbar_init(&bar_p_full[i], 4);
            nm_mbar_init(&bar_p_empty[i], 1);
        }
        nm_fence_barrier_init();
    }
    if (warp == 0) {
        nm_tmem_alloc(&tmem_slot, a.tmem_cols);
        nm_tmem_relinquish();
    } else {
        // 32-way replicated exp table: entry s of lane l at rep[s*32 + l]; one extra entry (a copy
        // of the last) so that input 0 of a table whose range ends at 0 needs no clamp
        const int n = a.n_exp;
        for (int i = threadIdx.x - 32; i < (n + 1) * 32; i += NSOFT) rep[i] = a.t_exp->kb[min(i >> 5, n - 1)];
    }
    nm_tc_fence_before();
    __syncthreads();
    nm_tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    volatile int* abortp = &abort_flag;
    nm_grid_launch_dependents();   // the next kernel may start its set-up
    nm_grid_dependency_wait();     // Q, K, V come from the previous kernel
    const int n_pchunks = L / 64;

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            // ---- loads: Q and K on one barrier, V on another
            nm_mbar_expect_tx(&bar_qk, (uint32_t)(BQ * ROWB + L * ROWB));
            nm_tma_load_3d(q_s, &tmQ, g * HD, qb * BQ, b, &bar_qk);
            for (int j = 0; j < L / 128; ++j) nm_tma_load_3d(k_s + (size_t)j * 128 * ROWB, &tmK, g * HD, j * 128, b, &bar_qk);
            nm_mbar_expect_tx(&bar_v, (uint32_t)(L * ROWB));
            for (int j = 0; j < L / 128; ++j) nm_tma_load_3d(v_s + (size_t)j * 128 * ROWB, &tmV, g * HD, j * 128, b, &bar_v);
            // ---- S = Q K^T, 128 keys per instruction group
            ok = nm_mbar_wait(&bar_qk, 0, abortp, a.status);
            if (ok) {
                nm_tc_fence_after();
                const uint64_t qdesc = nm_smem_desc_sw128(nm_smem_u32(q_s));
                for (int jc = 0; jc < L / 128; ++jc) {
                    const uint64_t kdesc = nm_smem_desc_sw128(nm_smem_u32(k_s + (size_t)jc * 128 * ROWB));
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        nm_mma_f16(tmem_base + (uint32_t)(jc * 128), qdesc + 2 * k, kdesc + 2 * k, IDESC_QK, k != 0);
                }
                nm_tc_commit(&bar_s);
                ok = nm_mbar_wait(&bar_v, 0, abortp, a.status);
            }
            // ---- O += P V, 64 keys per P buffer
            for (int c = 0; ok && c < n_pchunks; ++c) {
                const int buf = c % a.nbuf;
                ok = nm_mbar_wait(&bar_p_full[buf], (uint32_t)((c / a.nbuf) & 1), abortp, a.status);
                if (!ok) break;
                nm_tc_fence_after();
                const uint64_t pdesc = nm_smem_desc_sw128(nm_smem_u32(p_s + (size_t)buf * BQ * ROWB));
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    // V rows (keys) c*64 + 16k .. +15: two groups of 8 rows, 1024 bytes apart
                    const uint64_t vdesc = nm_smem_desc_sw128(nm_smem_u32(v_s + (size_t)(c * 64 + 16 * k) * ROWB));
                    nm_mma_f16(tmem_base + a.o_col, pdesc + 2 * k, vdesc, IDESC_PV, (c | k) != 0);
                }
                nm_tc_commit(&bar_p_empty[buf]);
            }
            if (ok) nm_tc_commit(&bar_o);
            if (!ok) {
                // bounded drain: pending copies and MMAs get time to finish before teardown
                long long t0 = clock64();
                while (!nm_mbar_try_wait(&bar_qk, 0) && clock64() - t0 < 200000000LL) {}
                while (!nm_mbar_try_wait(&bar_v, 0) && clock64() - t0 < 400000000LL) {}
                nm_tc_commit(&bar_drain);
                while (!nm_mbar_try_wait(&bar_drain, 0) && clock64() - t0 < 600000000LL) {}
            }
        }
    } else {
        const int q = warp & 3;
        const int h = (warp - 1) >> 2;
        const int row = q * 32 + lane;
        const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
        const float inv_h = a.t_exp->inv_h, off = a.t_exp->off, nm1 = (float)(a.n_exp - 1);
        // this lane's column of the replicated table, with the constant of the index trick folded in
        const uint32_t rep_lane = nm_smem_u32(rep) + (uint32_t)lane * 8u - 0x40000000u;
        int ok = 1;
        if (lane == 0) ok = nm_mbar_wait_relaxed(&bar_s, 0, abortp, a.status) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        float m = -INFINITY;
        if (ok) {
            (void)nm_mbar_try_wait(&bar_s, 0);
            nm_tc_fence_after();
            // ---- pass 1: maximum over this warp's chunks
#pragma unroll 1
            for (int c = h; c < n_pchunks; c += NH) {
                uint32_t r[64];
                nm_tmem_ld32_sync(t_row + (uint32_t)(c * 64), r);
                nm_tmem_ld32_sync(t_row + (uint32_t)(c * 64 + 32), r + 32);
                float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
                for (int i = 0; i < 64; i += 4) {
                    m0 = max3(m0, __uint_as_float(r[i]), __uint_as_float(r[i + 1]));
                    m1 = max3(m1, __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
                }
                m = max3(m, m0, m1);
            }
        }
        s_red[h][row] = m;
        asm volatile("bar.sync 1, %0;" ::"n"(NSOFT) : "memory");
#pragma unroll
        for (int i = 0; i < NH; ++i) m = fmaxf(m, s_red[i][row]);  // the FINAL row maximum
        asm volatile("bar.sync 1, %0;" ::"n"(NSOFT) : "memory");
        const float neg_ms = -(m * a.scale);
        float sum0 = 0.f, sum1 = 0.f, sum2 = 0.f, sum3 = 0.f;
        if (ok) {
            // ---- pass 2: e = PWL_exp(s - m), row sum, P tiles for the second MMA
#pragma unroll 1
            for (int c = h; c < n_pchunks; c += NH) {
                const int buf = c % a.nbuf;
                if (c >= a.nbuf) {
                    if (lane == 0) ok = nm_mbar_wait_relaxed(&bar_p_empty[buf], (uint32_t)(((c / a.nbuf) - 1) & 1), abortp, a.status) ? 1 : 0;
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) break;
                    (void)nm_mbar_try_wait(&bar_p_empty[buf], (uint32_t)(((c / a.nbuf) - 1) & 1));
                }
                const uint32_t prow = nm_smem_u32(p_s) + (uint32_t)(buf * BQ * ROWB + row * ROWB);
                uint32_t r[64];
                nm_tmem_ld32_sync(t_row + (uint32_t)(c * 64), r);
                nm_tmem_ld32_sync(t_row + (uint32_t)(c * 64 + 32), r + 32);
#pragma unroll
                for (int j = 0; j < 8; ++j) {  // 8 keys = one 16-byte chunk of the P row
                    float e[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float x = __fmaf_rn(__uint_as_float(r[j * 8 + i]), a.scale, neg_ms);
                        float u = fmaxf(__fmaf_rn(x, inv_h, off), 0.0f);
                        if (CLAMP_HI) u = fminf(u, nm1);
                        // floor(u) sits in the low mantissa bits after a round-down add of 1.5 * 2^23
                        const uint32_t bits = __float_as_uint(__fadd_rd(u, 12582912.0f));
                        float kk, bb;
                        asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(kk), "=f"(bb) : "r"((bits << 8) + rep_lane));
                        e[i] = __fmaf_rn(kk, x, bb);
                    }
                    sum0 += e[0] + e[4];
                    sum1 += e[1] + e[5];
                    sum2 += e[2] + e[6];
                    sum3 += e[3] + e[7];
                    // chunk index is XORed with the row (128-byte swizzle of the K-major P tile)
                    const uint32_t addr = prow + (uint32_t)((j ^ (row & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(AttnT<T>::pack(e[0], e[1])),
                                 "r"(AttnT<T>::pack(e[2], e[3])), "r"(AttnT<T>::pack(e[4], e[5])),
                                 "r"(AttnT<T>::pack(e[6], e[7]))
                                 : "memory");
                }
                nm_fence_proxy_async();  // generic-proxy writes of P become visible to the tensor core
                nm_tc_fence_before();
                __syncwarp();
                if (lane == 0) nm_mbar_arrive(&bar_p_full[buf]);
                __syncwarp();
            }
        }
        s_red[h][row] = (sum0 + sum1) + (sum2 + sum3);
        asm volatile("bar.sync 1, %0;" ::"n"(NSOFT) : "memory");
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < NH; ++i) sum += s_red[i][row];
        if (ok) {
            // ---- r = PWL_recip(sigma), then O * r; each warp group stores 64/NH of the 64 channels
            const int sr = nm_pwl_index(sum, a.t_rcp->inv_h, a.t_rcp->off, (float)(a.t_rcp->n - 1));
            const float2 kbr = a.t_rcp->kb[sr];
            const float rinv = __fmaf_rn(kbr.x, sum, kbr.y);
            if (lane == 0) ok = nm_mbar_wait_relaxed(&bar_o, 0, abortp, a.status) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (ok) {
                (void)nm_mbar_try_wait(&bar_o, 0);
                nm_tc_fence_after();
                constexpr int CH = HD / NH;  // channels per warp group: 16 or 32
                T* orow = reinterpret_cast<T*>(a.out) + ((size_t)b * L + (size_t)qb * BQ + row) * ((size_t)a.heads * HD) +
                          (size_t)g * HD + h * CH;
#pragma unroll
                for (int part = 0; part < CH / 16; ++part) {
                    uint32_t r[16];
                    tmem_ld16(t_row + a.o_col + (uint32_t)(h * CH + part * 16), r);
                    uint32_t w[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        w[i] = AttnT<T>::pack(__uint_as_float(r[2 * i]) * rinv, __uint_as_float(r[2 * i + 1]) * rinv);
                    reinterpret_cast<uint4*>(orow + part * 16)[0] = make_uint4(w[0], w[1], w[2], w[3]);
                    reinterpret_cast<uint4*>(orow + part * 16)[1] = make_uint4(w[4], w[5], w[6], w[7]);
                }
            }
        }
    }

    nm_tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        nm_tc_fence_after();
        nm_tmem_dealloc(tmem_base, a.tmem_cols);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [B][L][heads*64] view with token pitch stride_t and batch pitch stride_b (elements); box 64 x 128 x 1.
nm_status make_map(nm_ctx* ctx, CUtensorMap* m, const void* ptr, nm_dtype dt, const nm_attn_desc* d)
{
    CUtensorMapDataType t = dt == NM_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
    cuuint64_t gdim[3] = {(cuuint64_t)d->heads * HD, (cuuint64_t)d->L, (cuuint64_t)d->B};
    cuuint64_t gstr[2] = {(cuuint64_t)d->stride_t * 2, (cuuint64_t)d->stride_b * 2};
    cuuint32_t box[3] = {HD, 128, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = ((EncodeTiledFn)ctx->encode_tiled)(m, t, 3, const_cast<void*>(ptr), gdim, gstr, box, estr,
                                                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? NM_OK : NM_ERR_CUDA;
}

template <typename T, int NH, bool CLAMP_HI>
nm_status launch(nm_ctx* ctx, const nm_attn_desc* d, cudaStream_t st)
{
    AttnArgs a;
    a.B = d->B; a.L = d->L; a.heads = d->heads; a.scale = d->scale;
    a.t_exp = ctx->d_tables + d->exp_slot;
    a.t_rcp = ctx->d_tables + d->recip_slot;
    a.out = d->out;
    a.status = ctx->d_status;
    a.n_exp = ctx->h_tables[d->exp_slot].n;
    const int L = d->L;
    a.p_in_k = L >= 256 ? 1 : 0;
    a.nbuf = L >= 256 ? L / 128 : 2;
    if (L == 128) { a.tmem_cols = 256; a.o_col = 128; }
    else if (L == 512) { a.tmem_cols = 512; a.o_col = 0; }  // O reuses the first 64 columns of S
    else { a.tmem_cols = 512; a.o_col = (uint32_t)L; }
    const size_t tiles = (size_t)BQ * ROWB + 2 * (size_t)L * ROWB + (a.p_in_k ? 0 : (size_t)a.nbuf * BQ * ROWB);
    const size_t smem = tiles + (size_t)(a.n_exp + 1) * 32 * sizeof(float2) + 1024;
    if (smem > 227 * 1024 - 2048) return NM_ERR_UNSUPPORTED;

    CUtensorMap tmQ, tmK, tmV;
    nm_status s;
    if ((s = make_map(ctx, &tmQ, d->Q, d->dtype, d)) != NM_OK) return s;
    if ((s = make_map(ctx, &tmK, d->K, d->dtype, d)) != NM_OK) return s;
    if ((s = make_map(ctx, &tmV, d->V, d->dtype, d)) != NM_OK) return s;
    auto kern = attention_tc_kernel<T, NH, CLAMP_HI>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return NM_ERR_CUDA;
    const int64_t grid = (int64_t)d->B * d->heads * (L / BQ);
    if (grid > 0x7fffffffLL) return NM_ERR_SHAPE;
    NmLaunchScope scope(ctx, NM_KERNEL_ATTENTION_TC, 4.0 * (double)d->B * d->heads * (double)L * L * HD, st);
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(32 + 128 * NH);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = ctx->pdl ? 1 : 0;
    if (cudaLaunchKernelEx(&cfg, kern, tmQ, tmK, tmV, a) != cudaSuccess) return NM_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

template <typename T>
nm_status launch_sel(nm_ctx* ctx, const nm_attn_desc* d, cudaStream_t st)
{
    // the softmax input is never positive: a table whose range reaches 0 needs no upper clamp
    const bool clamp_hi = ctx->h_tables[d->exp_slot].x_max < 0.0f;
    if (d->L >= 256) return clamp_hi ? launch<T, 4, true>(ctx, d, st) : launch<T, 4, false>(ctx, d, st);
    return clamp_hi ? launch<T, 2, true>(ctx, d, st) : launch<T, 2, false>(ctx, d, st);
}

}  // namespace

bool nm_attention_tc_supported(const nm_attn_desc* d)
{
    if (d->dtype != NM_BF16 && d->dtype != NM_F16) return false;
    if (d->d != HD) return false;
    if (d->L % 128 != 0 || d->L < 128 || d->L > 512) return false;
    if ((d->stride_t * 2) % 16 != 0 || (d->stride_b * 2) % 16 != 0) return false;
    return true;
}

nm_status nm_launch_attention_tc(nm_ctx* ctx, const nm_attn_desc* d, cudaStream_t st)
{
    if (!nm_attention_tc_supported(d)) return NM_ERR_UNSUPPORTED;
    return d->dtype == NM_BF16 ? launch_sel<__nv_bfloat16>(ctx, d, st) : launch_sel<__half>(ctx, d, st);
}
