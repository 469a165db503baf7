// Linear operator with fused PWL epilogue on the 5th-generation tensor cores
// (Section 3.1: a linear operator is a matrix product plus matrix adds; Section 3.2:
// Y = X.K + B per element, K and B gathered by segment number).
//
//   out[m][j] = PWL( sum_c A[m][c]*W[j][c] * scale_j + bias[j] ) + residual[m][j]
//
// Persistent, warp-specialised kernel, one CTA per SM:
//   warp 0     TMA producer: 128 x 128-byte A tile and BN x 128-byte W tile per stage,
//              128-byte swizzle, multi-stage mbarrier ring
//   warp 1     tcgen05.mma issuer (one lane); accumulators live in tensor memory,
//              two buffers of BN columns so the epilogue of tile i overlaps the
//              main loop of tile i+1
//   warps 2-9  epilogue, two warps per tensor-memory lane quarter: tcgen05.ld -> bias/scale ->
//              segment index -> k*x+b from a per-lane replicated table in shared memory ->
//              residual -> store; the loads of the next 32-column chunk are in flight
//              while the current one is computed.
// The nonlinearity therefore costs no pass over HBM.
#include "nm_common.cuh"

namespace {

constexpr int BM = 128;
constexpr int ROW_BYTES = 128;  // bytes of K per tile row = one swizzle span
constexpr int A_BYTES = BM * ROW_BYTES;
constexpr int MAX_STAGES = 8;
constexpr int NUM_THREADS = 320;  // TMA warp, MMA warp, 8 epilogue warps

struct TcArgs {
    int64_t M, N, K;
    int64_t ldr, ldo;
    const float* bias;
    const void* residual;
    void* out;
    const NmTable* tab;
    float a_scale;
    const float* w_scale;
    float inv_out_scale;
    int32_t* acc_dump;
    int32_t* idx_dump;
    int* status;
    int num_n_tiles, num_tiles, num_k_blocks, stages, n_seg;
};

template <typename InT> struct TcIn;
template <> struct TcIn<__nv_bfloat16> {
    static constexpr uint32_t c_fmt = 1, ab_fmt = 1;
    static constexpr bool is_int = false;
};
template <> struct TcIn<__half> {
    static constexpr uint32_t c_fmt = 1, ab_fmt = 0;
    static constexpr bool is_int = false;
};
template <> struct TcIn<int8_t> {
    static constexpr uint32_t c_fmt = 2, ab_fmt = 1;
    static constexpr bool is_int = true;
};

template <typename OutT> __device__ __forceinline__ void store32(OutT* p, const float* v, float inv);
template <> __device__ __forceinline__ void store32<__nv_bfloat16>(__nv_bfloat16* p, const float* v, float)
{
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint4 raw;
        __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&raw);
#pragma unroll
        for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(v[q * 8 + 2 * i], v[q * 8 + 2 * i + 1]);
        reinterpret_cast<uint4*>(p)[q] = raw;
    }
}
template <> __device__ __forceinline__ void store32<__half>(__half* p, const float* v, float)
{
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint4 raw;
        __half2* h = reinterpret_cast<__half2*>(&raw);
#pragma unroll
        for (int i = 0; i < 4; ++i) h[i] = __floats2half2_rn(v[q * 8 + 2 * i], v[q * 8 + 2 * i + 1]);
        reinterpret_cast<uint4*>(p)[q] = raw;
    }
}
template <> __device__ __forceinline__ void store32<float>(float* p, const float* v, float)
{
#pragma unroll
    for (int q = 0; q < 8; ++q)
        reinterpret_cast<float4*>(p)[q] = make_float4(v[q * 4], v[q * 4 + 1], v[q * 4 + 2], v[q * 4 + 3]);
}
template <> __device__ __forceinline__ void store32<int8_t>(int8_t* p, const float* v, float inv)
{
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        uint4 raw;
        int8_t* e = reinterpret_cast<int8_t*>(&raw);
#pragma unroll
        for (int i = 0; i < 16; ++i) e[i] = nm_quant_i8(v[q * 16 + i], inv);
        reinterpret_cast<uint4*>(p)[q] = raw;
    }
}

template <typename OutT> __device__ __forceinline__ void store1(OutT* p, float v, float) { *p = NmType<OutT>::from_f(v); }
template <> __device__ __forceinline__ void store1<int8_t>(int8_t* p, float v, float inv) { *p = nm_quant_i8(v, inv); }

template <typename OutT> __device__ __forceinline__ void add_res32(const uint4* p, float* v)
{
    constexpr int PER = 16 / sizeof(OutT);
#pragma unroll
    for (int q = 0; q < 32 / PER; ++q) {
        uint4 raw = p[q];
        const OutT* e = reinterpret_cast<const OutT*>(&raw);
#pragma unroll
        for (int i = 0; i < PER; ++i) v[q * PER + i] += NmType<OutT>::to_f(e[i]);
    }
}
template <> __device__ __forceinline__ void add_res32<int8_t>(const uint4*, float*) {}
template <typename OutT> __device__ __forceinline__ float res1(const OutT* p) { return NmType<OutT>::to_f(*p); }
template <> __device__ __forceinline__ float res1<int8_t>(const int8_t*) { return 0.f; }

template <typename InT, typename OutT, int BN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
linear_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW, const TcArgs a)
{
    constexpr int B_BYTES = BN * ROW_BYTES;
    constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    constexpr int BK_ELEMS = ROW_BYTES / (int)sizeof(InT);
    constexpr uint32_t TMEM_COLS = 2 * BN;  // 512 or 256: a power of two
    constexpr uint32_t IDESC = nm_idesc(TcIn<InT>::c_fmt, TcIn<InT>::ab_fmt, 0, 0, BM, BN);

    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_full[MAX_STAGES];
    __shared__ uint64_t bar_empty[MAX_STAGES];
    __shared__ uint64_t bar_acc_full[2];
    __shared__ uint64_t bar_acc_empty[2];
    __shared__ uint64_t bar_drain;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    float2* rep = reinterpret_cast<float2*>(tiles + (size_t)a.stages * STAGE_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int stages = a.stages;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        nm_prefetch_tmap(&tmA);
        nm_prefetch_tmap(&tmW);
        for (int s = 0; s < stages; ++s) {
            nm_mbar_init(&bar_full[s], 1);
            nm_mbar_init(&bar_empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            nm_mbar_init(&bar_acc_full[b], 1);
            nm_mbar_init(&bar_acc_empty[b], 8);
        }
        nm_mbar_init(&bar_drain, 1);
        nm_fence_barrier_init();
    }
    if (warp == 1) {
        nm_tmem_alloc(&tmem_slot, TMEM_COLS);
        nm_tmem_relinquish();
    }
    if (a.tab) nm_table_replicate(rep, a.tab, a.n_seg, threadIdx.x, NUM_THREADS);
    nm_tc_fence_before();
    __syncthreads();
    nm_tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    volatile int* abortp = &abort_flag;

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            long long issued = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < a.num_tiles; tile += gridDim.x) {
                const int m0 = (tile / a.num_n_tiles) * BM;
                const int n0 = (tile % a.num_n_tiles) * BN;
                for (int kb = 0; kb < a.num_k_blocks; ++kb) {
                    if (!nm_mbar_wait(&bar_empty[stage], phase ^ 1u, abortp, a.status)) { ok = false; break; }
                    uint8_t* sa = tiles + (size_t)stage * STAGE_BYTES;
                    nm_mbar_expect_tx(&bar_full[stage], STAGE_BYTES);
                    nm_tma_load_2d(sa, &tmA, kb * BK_ELEMS, m0, &bar_full[stage]);
                    nm_tma_load_2d(sa + A_BYTES, &tmW, kb * BK_ELEMS, n0, &bar_full[stage]);
                    ++issued;
                    if (++stage == stages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // give the copies already issued a bounded time to land before the CTA retires
                for (int s = 0; s < stages; ++s) {
                    long long last = -1;  // last iteration that used stage s
                    if (issued > s) last = ((issued - 1 - s) / stages) * stages + s;
                    if (last < 0) continue;
                    const uint32_t par = (uint32_t)((last / stages) & 1);
                    long long t0 = clock64();
                    while (!nm_mbar_try_wait(&bar_full[s], par) && clock64() - t0 < 200000000LL) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int buf = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < a.num_tiles; tile += gridDim.x) {
                if (!nm_mbar_wait(&bar_acc_empty[buf], acc_phase ^ 1u, abortp, a.status)) { ok = false; break; }
                nm_tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                for (int kb = 0; kb < a.num_k_blocks; ++kb) {
                    if (!nm_mbar_wait(&bar_full[stage], phase, abortp, a.status)) { ok = false; break; }
                    nm_tc_fence_after();
                    const uint32_t sa = nm_smem_u32(tiles + (size_t)stage * STAGE_BYTES);
                    const uint64_t adesc = nm_smem_desc_sw128(sa);
                    const uint64_t bdesc = nm_smem_desc_sw128(sa + A_BYTES);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {  // 4 x 32 bytes of K per 128-byte row
                        const uint32_t accum = (kb | k) != 0 ? 1u : 0u;
                        if constexpr (TcIn<InT>::is_int) nm_mma_i8(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC, accum);
                        else nm_mma_f16(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC, accum);
                    }
                    nm_tc_commit(&bar_empty[stage]);  // smem stage reusable once these MMAs retire
                    if (++stage == stages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                nm_tc_commit(&bar_acc_full[buf]);
                buf ^= 1;
                if (buf == 0) acc_phase ^= 1u;
            }
            if (!ok) {
                nm_tc_commit(&bar_drain);
                long long t0 = clock64();
                while (!nm_mbar_try_wait(&bar_drain, 0) && clock64() - t0 < 200000000LL) {}
            }
        }
    } else {
        // ------------------------------------------------ epilogue (warps 2..9)
        // Two warps per tensor-memory lane quarter; each takes half of the tile's columns in
        // 32-column chunks.  The tensor-memory load and the residual load of chunk i+1 are in
        // flight while chunk i is computed and stored.
        const int q = warp & 3;              // lane quarter this warp may read
        const int half = (warp - 2) >> 2;    // which half of the columns
        constexpr int NCH = BN / 64;         // chunks per warp per tile
        constexpr int RV = 2 * (int)sizeof(OutT);  // 16-byte vectors of residual per 32 columns
        int buf = 0;
        uint32_t acc_phase = 0;
        const bool has_tab = a.tab != nullptr;
        const float inv_h = has_tab ? a.tab->inv_h : 0.f;
        const float off = has_tab ? a.tab->off : 0.f;
        const float nm1 = (float)(a.n_seg - 1);
        OutT* out = reinterpret_cast<OutT*>(a.out);
        const OutT* res = reinterpret_cast<const OutT*>(a.residual);
        for (int tile = blockIdx.x; tile < a.num_tiles; tile += gridDim.x) {
            const int m0 = (tile / a.num_n_tiles) * BM;
            const int n0 = (tile % a.num_n_tiles) * BN + half * (BN / 2);
            int ok = 1;
            if (lane == 0) ok = nm_mbar_wait(&bar_acc_full[buf], acc_phase, abortp, a.status) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            nm_tc_fence_after();
            const int64_t row = (int64_t)m0 + q * 32 + lane;
            const bool row_ok = row < a.M;
            const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + half * (BN / 2));
            uint32_t r[2][32];
            uint4 rs[2][RV];
            nm_tmem_ld32_async(t_addr, r[0]);
            if (res && row_ok && n0 + 32 <= a.N) {
#pragma unroll
                for (int v = 0; v < RV; ++v) rs[0][v] = __ldg(reinterpret_cast<const uint4*>(res + row * a.ldr + n0) + v);
            }
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                const int cur = c & 1;
                nm_tmem_ld_wait32(r[cur]);
                const int64_t col0 = (int64_t)n0 + c * 32;
                if (c + 1 < NCH) {
                    nm_tmem_ld32_async(t_addr + (uint32_t)((c + 1) * 32), r[cur ^ 1]);
                    if (res && row_ok && col0 + 64 <= a.N) {
#pragma unroll
                        for (int v = 0; v < RV; ++v)
                            rs[cur ^ 1][v] = __ldg(reinterpret_cast<const uint4*>(res + row * a.ldr + col0 + 32) + v);
                    }
                } else {
                    // this warp's share of the accumulator is in registers: hand the buffer back
                    nm_tc_fence_before();
                    __syncwarp();
                    if (lane == 0) nm_mbar_arrive(&bar_acc_empty[buf]);
                    __syncwarp();
                }
                // lanes beyond the last row / column skip the arithmetic but stay in the loop:
                // the tensor-memory loads need the whole warp
                if (row_ok && col0 < a.N) {
                    float v[32];
                    if (col0 + 32 <= a.N) {
                        if constexpr (TcIn<InT>::is_int) {
                            if (a.acc_dump) {
#pragma unroll
                                for (int i = 0; i < 32; i += 4)
                                    *reinterpret_cast<int4*>(a.acc_dump + row * a.N + col0 + i) =
                                        make_int4((int)r[cur][i], (int)r[cur][i + 1], (int)r[cur][i + 2], (int)r[cur][i + 3]);
                            }
#pragma unroll
                            for (int i = 0; i < 32; i += 4) {
                                const float4 ws = __ldg(reinterpret_cast<const float4*>(a.w_scale + col0 + i));
                                float4 bs = make_float4(0.f, 0.f, 0.f, 0.f);
                                if (a.bias) bs = __ldg(reinterpret_cast<const float4*>(a.bias + col0 + i));
                                v[i] = __fmaf_rn((float)(int)r[cur][i], a.a_scale * ws.x, bs.x);
                                v[i + 1] = __fmaf_rn((float)(int)r[cur][i + 1], a.a_scale * ws.y, bs.y);
                                v[i + 2] = __fmaf_rn((float)(int)r[cur][i + 2], a.a_scale * ws.z, bs.z);
                                v[i + 3] = __fmaf_rn((float)(int)r[cur][i + 3], a.a_scale * ws.w, bs.w);
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[cur][i]);
                            if (a.bias) {
#pragma unroll
                                for (int i = 0; i < 32; i += 4) {
                                    const float4 bs = __ldg(reinterpret_cast<const float4*>(a.bias + col0 + i));
                                    v[i] += bs.x; v[i + 1] += bs.y; v[i + 2] += bs.z; v[i + 3] += bs.w;
                                }
                            }
                        }
                        if (has_tab) {
                            if (a.idx_dump) {
#pragma unroll
                                for (int i = 0; i < 32; ++i) {
                                    int s;
                                    v[i] = nm_pwl_eval_rep(rep, lane, v[i], inv_h, off, nm1, &s);
                                    a.idx_dump[row * a.N + col0 + i] = s;
                                }
                            } else {
#pragma unroll
                                for (int i = 0; i < 32; ++i) v[i] = nm_pwl_eval_rep(rep, lane, v[i], inv_h, off, nm1);
                            }
                        }
                        if (res) add_res32<OutT>(rs[cur], v);
                        store32<OutT>(out + row * a.ldo + col0, v, a.inv_out_scale);
                    } else {
                        // ragged right edge: element by element
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const int64_t col = col0 + i;
                            if (col >= a.N) continue;
                            float x;
                            const float bj = a.bias ? a.bias[col] : 0.f;
                            if constexpr (TcIn<InT>::is_int) {
                                if (a.acc_dump) a.acc_dump[row * a.N + col] = (int)r[cur][i];
                                x = __fmaf_rn((float)(int)r[cur][i], a.a_scale * a.w_scale[col], bj);
                            } else {
                                x = __uint_as_float(r[cur][i]) + bj;
                            }
                            if (has_tab) {
                                int s;
                                x = nm_pwl_eval_rep(rep, lane, x, inv_h, off, nm1, &s);
                                if (a.idx_dump) a.idx_dump[row * a.N + col] = s;
                            }
                            if (res) x += res1<OutT>(res + row * a.ldr + col);
                            store1<OutT>(out + row * a.ldo + col, x, a.inv_out_scale);
                        }
                    }
                }
                __syncwarp();
            }
            buf ^= 1;
            if (buf == 0) acc_phase ^= 1u;
        }
    }


    // ---------------------------------------------------- teardown (all paths)
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

// 2-D K-contiguous matrix [rows, cols] with row pitch ld (elements); box = 128 bytes x box_rows.
nm_status make_tmap(nm_ctx* ctx, CUtensorMap* m, const void* base, nm_dtype dt, int64_t rows, int64_t cols,
                    int64_t ld, int box_rows)
{
    const size_t es = nm_dtype_size(dt);
    CUtensorMapDataType t = dt == NM_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                            : dt == NM_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                           : CU_TENSOR_MAP_DATA_TYPE_UINT8;
    cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t gstr[1] = {(cuuint64_t)ld * es};
    cuuint32_t box[2] = {(cuuint32_t)(ROW_BYTES / es), (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = ((EncodeTiledFn)ctx->encode_tiled)(m, t, 2, const_cast<void*>(base), gdim, gstr, box, estr,
                                                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? NM_OK : NM_ERR_CUDA;
}

template <typename InT, typename OutT, int BN>
nm_status launch(nm_ctx* ctx, const nm_linear_desc* d, cudaStream_t st)
{
    constexpr int STAGE_BYTES = A_BYTES + BN * ROW_BYTES;
    TcArgs a;
    a.M = d->M; a.N = d->N; a.K = d->K; a.ldr = d->ldr; a.ldo = d->ldo;
    a.bias = d->bias; a.residual = d->residual; a.out = d->out;
    a.tab = d->slot == NM_SLOT_NONE ? nullptr : ctx->d_tables + d->slot;
    a.n_seg = d->slot == NM_SLOT_NONE ? 0 : ctx->h_tables[d->slot].n;
    a.a_scale = d->a_scale; a.w_scale = d->w_scale; a.inv_out_scale = d->inv_out_scale;
    a.acc_dump = d->acc_dump; a.idx_dump = d->idx_dump;
    a.status = ctx->d_status;
    const int bk = ROW_BYTES / (int)sizeof(InT);
    const int64_t m_tiles = (d->M + BM - 1) / BM;
    a.num_n_tiles = (int)((d->N + BN - 1) / BN);
    if (m_tiles * a.num_n_tiles > 0x7fffffffLL) return NM_ERR_SHAPE;
    a.num_tiles = (int)(m_tiles * a.num_n_tiles);
    a.num_k_blocks = (int)((d->K + bk - 1) / bk);
    const size_t table_bytes = (size_t)a.n_seg * 32 * sizeof(float2);
    const size_t budget = 227 * 1024 - 1024 /*alignment slack*/ - 1024 /*static*/ - table_bytes;
    int stages = (int)(budget / STAGE_BYTES);
    if (stages > MAX_STAGES) stages = MAX_STAGES;
    if (stages < 2) return NM_ERR_UNSUPPORTED;
    a.stages = stages;
    const size_t smem = (size_t)stages * STAGE_BYTES + table_bytes + 1024;

    CUtensorMap tmA, tmW;
    nm_status s = make_tmap(ctx, &tmA, d->A, d->in_dtype, d->M, d->K, d->lda, BM);
    if (s != NM_OK) return s;
    s = make_tmap(ctx, &tmW, d->W, d->in_dtype, d->N, d->K, d->ldw, BN);
    if (s != NM_OK) return s;

    auto kern = linear_tc_kernel<InT, OutT, BN>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return NM_ERR_CUDA;
    const int grid = a.num_tiles < ctx->sm_count ? a.num_tiles : ctx->sm_count;
    NmLaunchScope scope(ctx, NM_KERNEL_LINEAR_TC, 2.0 * (double)d->M * (double)d->N * (double)d->K, st);
    kern<<<grid, NUM_THREADS, smem, st>>>(tmA, tmW, a);
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

template <typename InT, typename OutT>
nm_status launch_bn(nm_ctx* ctx, const nm_linear_desc* d, cudaStream_t st)
{
    if (d->N % 256 == 0 || d->N >= 1024) return launch<InT, OutT, 256>(ctx, d, st);
    return launch<InT, OutT, 128>(ctx, d, st);
}

}  // namespace

bool nm_linear_tc_supported(const nm_linear_desc* d)
{
    if (d->in_dtype == NM_F32) return false;
    const size_t es = nm_dtype_size(d->in_dtype);
    if (d->M < 1 || d->N < 8 || d->K < 1) return false;
    if ((d->K * es) % 16 != 0) return false;  // TMA: global extents and pitches in 16-byte units
    if (d->N % 4 != 0) return false;          // vector dumps / bias loads
    if (d->in_dtype == NM_I8) return d->out_dtype == NM_BF16 || d->out_dtype == NM_F32 || d->out_dtype == NM_I8;
    return d->out_dtype == d->in_dtype;
}

nm_status nm_launch_linear_tc(nm_ctx* ctx, const nm_linear_desc* d, cudaStream_t st)
{
    if (!nm_linear_tc_supported(d)) return NM_ERR_UNSUPPORTED;
    switch (d->in_dtype) {
    case NM_BF16: return launch_bn<__nv_bfloat16, __nv_bfloat16>(ctx, d, st);
    case NM_F16: return launch_bn<__half, __half>(ctx, d, st);
    case NM_I8:
        if (d->out_dtype == NM_BF16) return launch_bn<int8_t, __nv_bfloat16>(ctx, d, st);
        if (d->out_dtype == NM_F32) return launch_bn<int8_t, float>(ctx, d, st);
        return launch_bn<int8_t, int8_t>(ctx, d, st);
    default: return NM_ERR_UNSUPPORTED;
    }
}
