// Fused attention with PWL softmax, streaming variant: two CTAs per SM.
//
// Same function as attention_tc.cu (Section 3.1: attention is a linear operator; Section 3.2.2:
// exp and 1/x as PWL tables), per query row
//     s_j = scale*<q,k_j>;  m = max_j s_j;  e_j = PWL_exp(s_j - m);  sigma = sum_j e_j;
//     o = PWL_recip(sigma) * sum_j e_j v_j
// with m the FINAL row maximum (a PWL exponential is not multiplicative, so there is no
// running-maximum rescaling).  Instead of keeping the whole 128 x L score block in tensor memory,
// this kernel computes Q K^T TWICE: a first sweep over the keys only for the row maximum, a second
// sweep for the exponentials.  The tensor pipe is idle most of the time in this ALU-bound kernel, so
// the second Q K^T is free, and the footprint drops to 256 tensor-memory columns and ~105 KB of
// shared memory: two CTAs fit on an SM and one CTA's loads, MMAs and barriers overlap the other's
// arithmetic.  Any L that is a multiple of 128 is supported.
//
//   warp 0      TMA producer: Q once; K and V in 64-key chunks through a 6-stage ring, in exactly
//               the order the MMA warp consumes them (K0..Kn-1, then K0, K1, V0, K2, V1, ...)
//   warp 1      tcgen05.mma issuer: S chunk = Q K_c^T (128 x 64) into one of two tensor-memory
//               buffers; in the second sweep also O += P_c V_c (V as an MN-major operand)
//   warps 2-9   softmax, two per tensor-memory lane quarter, each owning 32 of a chunk's 64
//               columns: tcgen05.ld, row maximum (sweep 1); PWL exp, row sum, bf16 P tile in the
//               swizzled K-major layout (sweep 2); PWL reciprocal, scaling, store.
#include <string.h>

#include "nm_common.cuh"

namespace {

constexpr int BQ = 128;    // query rows per CTA
constexpr int HD = 64;     // head dimension
constexpr int CK = 64;     // keys per chunk
constexpr int ROWB = 128;  // bytes per tile row (64 x 16-bit)
constexpr int NS = 6;      // K/V ring stages
constexpr int STAGE = CK * ROWB;      // 8 KB
constexpr int PBUF = BQ * ROWB;       // 16 KB
constexpr int NTHREADS = 320;
constexpr int NSOFT = 256;

struct SArgs {
    int B, L, heads;
    float scale;
    const NmTable* t_exp;
    const NmTable* t_rcp;
    void* out;
    int* status;
    int n_exp;
};

template <typename T> struct AT;
template <> struct AT<__nv_bfloat16> {
    static constexpr uint32_t fmt = 1;
    static __device__ __forceinline__ uint32_t pack(float a, float b)
    {
        __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
        return *reinterpret_cast<uint32_t*>(&h);
    }
};
template <> struct AT<__half> {
    static constexpr uint32_t fmt = 0;
    static __device__ __forceinline__ uint32_t pack(float a, float b)
    {
        __half2 h = __floats2half2_rn(a, b);
        return *reinterpret_cast<uint32_t*>(&h);
    }
};

__device__ __forceinline__ float max3f(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

template <typename T, bool CLAMP_HI>
__global__ void __launch_bounds__(NTHREADS, 2)
attention_stream_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                        const __grid_constant__ CUtensorMap tmV, const SArgs a)
{
    constexpr uint32_t IDESC_QK = nm_idesc(1, AT<T>::fmt, 0, 0, BQ, CK);   // S chunk: 128 x 64
    constexpr uint32_t IDESC_PV = nm_idesc(1, AT<T>::fmt, 0, 1, BQ, HD);   // O: 128 x 64, V MN-major
    constexpr uint32_t TMEM_COLS = 256;                                     // S0 | S1 | O | unused
    constexpr uint32_t O_COL = 128;

    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_q, bar_o, bar_drain;
    __shared__ uint64_t bar_kv_full[NS], bar_kv_empty[NS];
    __shared__ uint64_t bar_s_full[2], bar_s_empty[2], bar_p_full[2], bar_p_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ float s_red[2][BQ];

    const int L = a.L;
    const int n = L / CK;  // chunks
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* q_s = base;                       // 16 KB
    uint8_t* ring = q_s + BQ * ROWB;           // NS x 8 KB
    uint8_t* p_s = ring + NS * STAGE;          // 2 x 16 KB
    float2* rep = reinterpret_cast<float2*>(p_s + 2 * PBUF);   // (n_exp + 1) x 16 copies

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
        nm_mbar_init(&bar_q, 1);
        nm_mbar_init(&bar_o, 1);
        nm_mbar_init(&bar_drain, 1);
        for (int i = 0; i < NS; ++i) {
            nm_mbar_init(&bar_kv_full[i], 1);
            nm_mbar_init(&bar_kv_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            nm_mbar_init(&bar_s_full[i], 1);
            nm_mbar_init(&bar_s_empty[i], 8);
            nm_mbar_init(&bar_p_full[i], 8);
            nm_mbar_init(&bar_p_empty[i], 1);
        }
        nm_fence_barrier_init();
    }
    if (warp == 1) {
        nm_tmem_alloc(&tmem_slot, TMEM_COLS);
        nm_tmem_relinquish();
    }
    if (warp >= 2) {
        // 16-way replicated exp table: entry s, copy c at rep[s*16 + c].  A 64-bit warp load is served
        // half a warp at a time, so 16 copies already make arbitrary lookups conflict-free.  One extra
        // entry (a copy of the last) lets input 0 of a table whose range ends at 0 go unclamped.
        const int ne = a.n_exp;
        for (int i = threadIdx.x - 64; i < (ne + 1) * 16; i += NSOFT) rep[i] = a.t_exp->kb[min(i >> 4, ne - 1)];
    }
    nm_tc_fence_before();
    __syncthreads();
    nm_tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    volatile int* abortp = &abort_flag;
    nm_grid_launch_dependents();   // the next kernel may start its set-up
    nm_grid_dependency_wait();     // Q, K, V come from the previous kernel

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            nm_mbar_expect_tx(&bar_q, BQ * ROWB);
            nm_tma_load_3d(q_s, &tmQ, g * HD, qb * BQ, b, &bar_q);
            auto push = [&](const CUtensorMap* tm, int chunk) {
                if (!ok) return;
                // the ring is deep and this warp shares its scheduler with softmax warps: sleep between polls
                if (!nm_mbar_wait_relaxed<200>(&bar_kv_empty[stage], phase ^ 1u, abortp, a.status)) { ok = false; return; }
                nm_mbar_expect_tx(&bar_kv_full[stage], STAGE);
                nm_tma_load_3d(ring + (size_t)stage * STAGE, tm, g * HD, chunk * CK, b, &bar_kv_full[stage]);
                if (++stage == NS) { stage = 0; phase ^= 1u; }
            };
            for (int c = 0; c < n; ++c) push(&tmK, c);        // sweep 1
            push(&tmK, 0);                                     // sweep 2
            for (int c = 0; c < n; ++c) {
                if (c + 1 < n) push(&tmK, c + 1);
                push(&tmV, c);
            }
            if (!ok) {
                long long t0 = clock64();  // bounded pause: copies in flight land before teardown
                while (clock64() - t0 < 4000000LL) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            uint32_t t = 0;   // S chunks issued so far; chunk t uses buffer t & 1 for the (t >> 1)-th time (n is even)
            bool ok = nm_mbar_wait_relaxed<20>(&bar_q, 0, abortp, a.status);
            const uint64_t qdesc = nm_smem_desc_sw128(nm_smem_u32(q_s));
            auto qk = [&](int c) {   // S[c & 1] = Q K_c^T
                if (!ok) return;
                const int sb = c & 1;
                if (!nm_mbar_wait_relaxed<20>(&bar_s_empty[sb], ((t >> 1) & 1u) ^ 1u, abortp, a.status)) { ok = false; return; }
                if (!nm_mbar_wait_relaxed<20>(&bar_kv_full[stage], phase, abortp, a.status)) { ok = false; return; }
                nm_tc_fence_after();
                const uint64_t kdesc = nm_smem_desc_sw128(nm_smem_u32(ring + (size_t)stage * STAGE));
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    nm_mma_f16(tmem_base + (uint32_t)(sb * CK), qdesc + 2 * k, kdesc + 2 * k, IDESC_QK, k != 0);
                nm_tc_commit(&bar_kv_empty[stage]);
                nm_tc_commit(&bar_s_full[sb]);
                ++t;
                if (++stage == NS) { stage = 0; phase ^= 1u; }
            };
            for (int c = 0; c < n; ++c) qk(c);   // sweep 1: scores for the row maximum
            qk(0);                               // sweep 2
            for (int c = 0; c < n && ok; ++c) {
                if (c + 1 < n) qk(c + 1);
                if (!ok) break;
                const int pb = c & 1;
                if (!nm_mbar_wait_relaxed<20>(&bar_p_full[pb], (uint32_t)((c >> 1) & 1), abortp, a.status)) { ok = false; break; }
                if (!nm_mbar_wait_relaxed<20>(&bar_kv_full[stage], phase, abortp, a.status)) { ok = false; break; }
                nm_tc_fence_after();
                const uint64_t pdesc = nm_smem_desc_sw128(nm_smem_u32(p_s + (size_t)pb * PBUF));
                const uint32_t v_addr = nm_smem_u32(ring + (size_t)stage * STAGE);
#pragma unroll
                for (int k = 0; k < 4; ++k)   // V rows (keys) 16k..16k+15: two groups of 8 rows, 1024 bytes apart
                    nm_mma_f16(tmem_base + O_COL, pdesc + 2 * k, nm_smem_desc_sw128(v_addr + (uint32_t)(16 * k * ROWB)),
                               IDESC_PV, (c | k) != 0);
                nm_tc_commit(&bar_kv_empty[stage]);
                nm_tc_commit(&bar_p_empty[pb]);
                if (++stage == NS) { stage = 0; phase ^= 1u; }
            }
            if (ok) nm_tc_commit(&bar_o);
            else {
                nm_tc_commit(&bar_drain);
                long long t0 = clock64();
                while (!nm_mbar_try_wait(&bar_drain, 0) && clock64() - t0 < 200000000LL) {}
            }
        }
    } else {
        // ------------------------------------------------ softmax warps
        const int q = warp & 3;
        const int h = (warp - 2) >> 2;
        const int row = q * 32 + lane;
        const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(h * 32);
        const float inv_h = a.t_exp->inv_h, off = a.t_exp->off, nm1 = (float)(a.n_exp - 1);
        // this lane's copy of the replicated table, with the constant of the index trick folded in:
        // (bits << 7) = 0xA0000000 + s*128 (mod 2^32) for bits = 0x4B400000 + s
        const uint32_t rep_lane = nm_smem_u32(rep) + (uint32_t)(lane & 15) * 8u - 0xA0000000u;
        int ok = 1;
        uint32_t t = 0;   // S chunks consumed so far; chunk t sits in buffer t & 1, its (t >> 1)-th use (n is even)
        // waits for the next S chunk, loads this warp's 32 columns, hands the buffer back
        auto load_s = [&](int sb, uint32_t* r) {
            const uint32_t par = (t >> 1) & 1u;
            if (lane == 0 && ok) ok = nm_mbar_wait_relaxed(&bar_s_full[sb], par, abortp, a.status) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (ok) {
                (void)nm_mbar_try_wait(&bar_s_full[sb], par);
                nm_tc_fence_after();
                nm_tmem_ld32_async(t_row + (uint32_t)(sb * CK), r);
                nm_tmem_ld_wait32(r);
                nm_tc_fence_before();
                __syncwarp();
                if (lane == 0) nm_mbar_arrive(&bar_s_empty[sb]);
                __syncwarp();
            }
            ++t;
        };
        // ---- sweep 1: the final row maximum
        float m = -INFINITY;
#pragma unroll 1
        for (int c = 0; c < n; ++c) {
            uint32_t r[32];
            load_s(c & 1, r);
            if (ok) {
                float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    m0 = max3f(m0, __uint_as_float(r[i]), __uint_as_float(r[i + 1]));
                    m1 = max3f(m1, __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
                }
                m = max3f(m, m0, m1);
            }
        }
        s_red[h][row] = m;
        asm volatile("bar.sync 1, %0;" ::"n"(NSOFT) : "memory");
        m = fmaxf(s_red[0][row], s_red[1][row]);
        asm volatile("bar.sync 1, %0;" ::"n"(NSOFT) : "memory");
        const float neg_ms = -(m * a.scale);
        float sum0 = 0.f, sum1 = 0.f, sum2 = 0.f, sum3 = 0.f;
        // ---- sweep 2: e = PWL_exp(s - m), row sum, P tiles
#pragma unroll 1
        for (int c = 0; c < n; ++c) {
            uint32_t r[32];
            load_s(c & 1, r);
            const int pb = c & 1;
            if (c >= 2 && ok) {
                const uint32_t par = (uint32_t)(((c >> 1) - 1) & 1);
                if (lane == 0) ok = nm_mbar_wait_relaxed(&bar_p_empty[pb], par, abortp, a.status) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (ok) (void)nm_mbar_try_wait(&bar_p_empty[pb], par);
            }
            if (ok) {
                const uint32_t prow = nm_smem_u32(p_s) + (uint32_t)(pb * PBUF + row * ROWB);
#pragma unroll
                for (int j = 0; j < 4; ++j) {   // 8 keys = one 16-byte chunk of the P row
                    float e[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float x = __fmaf_rn(__uint_as_float(r[j * 8 + i]), a.scale, neg_ms);
                        float u = fmaxf(__fmaf_rn(x, inv_h, off), 0.0f);
                        if (CLAMP_HI) u = fminf(u, nm1);
                        // floor(u) sits in the low mantissa bits after a round-down add of 1.5 * 2^23
                        const uint32_t bits = __float_as_uint(__fadd_rd(u, 12582912.0f));
                        float kk, bb;
                        asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(kk), "=f"(bb) : "r"((bits << 7) + rep_lane));
                        e[i] = __fmaf_rn(kk, x, bb);
                    }
                    sum0 += e[0] + e[4];
                    sum1 += e[1] + e[5];
                    sum2 += e[2] + e[6];
                    sum3 += e[3] + e[7];
                    // chunk index is XORed with the row (128-byte swizzle of the K-major P tile)
                    const uint32_t addr = prow + (uint32_t)(((h * 4 + j) ^ (row & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(AT<T>::pack(e[0], e[1])),
                                 "r"(AT<T>::pack(e[2], e[3])), "r"(AT<T>::pack(e[4], e[5])), "r"(AT<T>::pack(e[6], e[7]))
                                 : "memory");
                }
                nm_fence_proxy_async();   // generic-proxy writes of P become visible to the tensor core
                nm_tc_fence_before();
                __syncwarp();
                if (lane == 0) nm_mbar_arrive(&bar_p_full[pb]);
                __syncwarp();
            }
        }
        s_red[h][row] = (sum0 + sum1) + (sum2 + sum3);
        asm volatile("bar.sync 1, %0;" ::"n"(NSOFT) : "memory");
        const float sum = s_red[0][row] + s_red[1][row];
        if (ok) {
            // ---- r = PWL_recip(sigma), then O * r; each half stores 32 of the 64 channels
            const int sr = nm_pwl_index(sum, a.t_rcp->inv_h, a.t_rcp->off, (float)(a.t_rcp->n - 1));
            const float2 kbr = a.t_rcp->kb[sr];
            const float rinv = __fmaf_rn(kbr.x, sum, kbr.y);
            if (lane == 0) ok = nm_mbar_wait_relaxed(&bar_o, 0, abortp, a.status) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (ok) {
                (void)nm_mbar_try_wait(&bar_o, 0);
                nm_tc_fence_after();
                T* orow = reinterpret_cast<T*>(a.out) + ((size_t)b * L + (size_t)qb * BQ + row) * ((size_t)a.heads * HD) +
                          (size_t)g * HD + h * 32;
                uint32_t r[32];
                nm_tmem_ld32_async(tmem_base + ((uint32_t)(q * 32) << 16) + O_COL + (uint32_t)(h * 32), r);
                nm_tmem_ld_wait32(r);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint32_t w[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        w[i] = AT<T>::pack(__uint_as_float(r[j * 8 + 2 * i]) * rinv, __uint_as_float(r[j * 8 + 2 * i + 1]) * rinv);
                    reinterpret_cast<uint4*>(orow)[j] = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        }
    }

    nm_tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        nm_tc_fence_after();
        nm_tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [B][L][heads*64] view with token pitch stride_t and batch pitch stride_b (elements); box 64 x rows x 1.
nm_status make_map(nm_ctx* ctx, CUtensorMap* m, const void* ptr, nm_dtype dt, const nm_attn_desc* d, int rows)
{
    CUtensorMapDataType t = dt == NM_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
    cuuint64_t gdim[3] = {(cuuint64_t)d->heads * HD, (cuuint64_t)d->L, (cuuint64_t)d->B};
    cuuint64_t gstr[2] = {(cuuint64_t)d->stride_t * 2, (cuuint64_t)d->stride_b * 2};
    cuuint32_t box[3] = {HD, (cuuint32_t)rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = ((EncodeTiledFn)ctx->encode_tiled)(m, t, 3, const_cast<void*>(ptr), gdim, gstr, box, estr,
                                                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? NM_OK : NM_ERR_CUDA;
}

template <typename T, bool CLAMP_HI>
nm_status launch(nm_ctx* ctx, const nm_attn_desc* d, cudaStream_t st)
{
    SArgs a;
    a.B = d->B; a.L = d->L; a.heads = d->heads; a.scale = d->scale;
    a.t_exp = ctx->d_tables + d->exp_slot;
    a.t_rcp = ctx->d_tables + d->recip_slot;
    a.out = d->out;
    a.status = ctx->d_status;
    a.n_exp = ctx->h_tables[d->exp_slot].n;
    const size_t smem = (size_t)BQ * ROWB + (size_t)NS * STAGE + 2 * (size_t)PBUF + (size_t)(a.n_exp + 1) * 16 * sizeof(float2) + 1024;
    if (smem > 227 * 1024 - 2048) return NM_ERR_UNSUPPORTED;   // an exp table too large to replicate
    CUtensorMap tmQ, tmK, tmV;
    nm_status s;
    if ((s = make_map(ctx, &tmQ, d->Q, d->dtype, d, BQ)) != NM_OK) return s;
    if ((s = make_map(ctx, &tmK, d->K, d->dtype, d, CK)) != NM_OK) return s;
    if ((s = make_map(ctx, &tmV, d->V, d->dtype, d, CK)) != NM_OK) return s;
    auto kern = attention_stream_kernel<T, CLAMP_HI>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return NM_ERR_CUDA;
    const int64_t grid = (int64_t)d->B * d->heads * (d->L / BQ);
    if (grid > 0x7fffffffLL) return NM_ERR_SHAPE;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = ctx->pdl ? 1 : 0;
    NmLaunchScope scope(ctx, NM_KERNEL_ATTENTION_TC, 4.0 * (double)d->B * d->heads * (double)d->L * d->L * HD, st);
    if (cudaLaunchKernelEx(&cfg, kern, tmQ, tmK, tmV, a) != cudaSuccess) return NM_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

}  // namespace

bool nm_attention_stream_supported(const nm_attn_desc* d)
{
    if (d->dtype != NM_BF16 && d->dtype != NM_F16) return false;
    if (d->d != HD) return false;
    if (d->L % 128 != 0 || d->L < 128) return false;
    if ((d->stride_t * 2) % 16 != 0 || (d->stride_b * 2) % 16 != 0) return false;
    return true;
}

nm_status nm_launch_attention_stream(nm_ctx* ctx, const nm_attn_desc* d, cudaStream_t st)
{
    if (!nm_attention_stream_supported(d)) return NM_ERR_UNSUPPORTED;
    // the softmax input is never positive: a table whose range reaches 0 needs no upper clamp
    const bool clamp_hi = ctx->h_tables[d->exp_slot].x_max < 0.0f;
    if (d->dtype == NM_BF16)
        return clamp_hi ? launch<__nv_bfloat16, true>(ctx, d, st) : launch<__nv_bfloat16, false>(ctx, d, st);
    return clamp_hi ? launch<__half, true>(ctx, d, st) : launch<__half, false>(ctx, d, st);
}
