// Linear operator with fused PWL epilogue on the 5th-generation tensor cores
// (Section 3.1: a linear operator -- a fully connected layer, a convolution -- is a matrix product
// plus matrix adds; Section 3.2: Y = X.K + B per element, K and B gathered by segment number).
//
//   out[m][j] = PWL( sum_c A[m][c]*W[j][c] * scale_j + bias[j] ) + residual[m][j]
//
// Persistent, warp-specialised kernel, one CTA per SM:
//   warp 0     TMA producer: 128 x 128-byte A tile and W tile per stage, 128-byte swizzle,
//              multi-stage mbarrier ring
//   warp 1     tcgen05.mma issuer (one lane); accumulators live in tensor memory, two
//              buffers of BN columns so the epilogue of tile i overlaps the main loop
//              of tile i+1
//   warps 2-9  epilogue, two warps per tensor-memory lane quarter.  Per 32-column chunk:
//              tcgen05.ld -> bias/scale -> segment index
//              -> k*x+b from a per-lane replicated table in shared memory -> residual.
//              Results are staged in shared memory (32 rows x 128 bytes per warp, 128-byte
//              swizzle) and leave with one TMA store per group, so global writes are whole
//              lines; the residual arrives the same way through a TMA load that is issued
//              one group ahead.
// The nonlinearity therefore costs no pass over HBM.
//
// BN = 256, 128 or 64 columns per tile (the MMA's N): narrow layers get a narrow tile instead of
//   multiplying zero-filled weight rows.  With BN = 64 the two warps of a lane quarter do not split
//   the tile's columns but take alternate tiles (each warp always reads the same accumulator buffer).
// TWO = false: one CTA per 128 x BN tile (tcgen05 cta_group::1).
// TWO = true:  a cluster of two CTAs per 256 x BN tile (cta_group::2): each CTA loads its
//   own 128 rows of A and its own BN/2 rows of W, the leader CTA issues one MMA over both,
//   and each CTA's tensor memory receives its 128 x BN half of the accumulator.
// CONV = true: A is not a matrix in memory but an NHWC activation, and the kernel is an implicit
//   GEMM convolution: a tile's 128 rows are a TW x TH patch of output pixels of NB images, and the
//   K-block of filter tap (ky, kx) and channel block cb is ONE 4-D TMA box of the activation itself,
//   shifted by the tap (and strided for a strided convolution); coordinates outside the image read
//   zeros, which is the convolution's padding.  Nothing is gathered into memory first.  Output and
//   residual tiles are 4-D boxes of the NHWC output in the same way.
#pragma once
#include <string.h>

#include "nm_common.cuh"

namespace nm_tc {

constexpr int BM = 128;
constexpr int ROW_BYTES = 128;  // bytes of K per tile row = one swizzle span
constexpr int A_BYTES = BM * ROW_BYTES;
constexpr int MAX_STAGES = 8;
constexpr int NUM_THREADS = 320;  // TMA warp, MMA warp, 8 epilogue warps
constexpr int NUM_EPI_WARPS = 8;
constexpr int STAGE_BUF = 32 * 128;  // one staging buffer: 32 rows x 128 bytes

// How a tile's 128 rows map onto the NHWC tensors of a convolution (CONV kernels only).
struct ConvDev {
    int tiles_x, tiles_y;   // patches per output row / column of an image
    int TW, TH, NB;         // patch: TW x TH output pixels of NB images; TW*TH*NB = 128, all powers of two
    int sw, sh, pw, ph;     // tap (ky, kx) of output pixel (oy, ox) reads input (oy*sh - ph + ky, ox*sw - pw + kx)
    int kw_eff, cblocks;    // K-block kb = (ky*kw_eff + kx)*cblocks + cb; 64 channels per block
    int Ho, Nimg;           // output rows per image, images
    int dw;                 // nonzero: "depthwise" form for pooling as a GEMM: column tile nt (64 channels) reads channel
                            // block nt of the activation at every tap and multiplies by ONE constant 64 x 64 matrix
};

struct TcArgs {
    int64_t M, N, K;
    const float* bias;
    int has_res;
    int res_first;  // residual is added before the table instead of after
    const NmTable* tab;
    float a_scale;
    const float* w_scale;
    float inv_out_scale;
    int32_t* acc_dump;
    int32_t* idx_dump;
    int* status;
    int num_n_tiles, num_tiles, num_k_blocks, stages, n_seg;
    ConvDev cv;
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

// 32 fp32 values -> 32*sizeof(OutT)/4 packed words
template <typename OutT> __device__ __forceinline__ void pack32(const float* v, uint32_t* w, float inv);
template <> __device__ __forceinline__ void pack32<__nv_bfloat16>(const float* v, uint32_t* w, float)
{
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t*>(&h);
    }
}
template <> __device__ __forceinline__ void pack32<__half>(const float* v, uint32_t* w, float)
{
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        __half2 h = __floats2half2_rn(v[2 * i], v[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t*>(&h);
    }
}
template <> __device__ __forceinline__ void pack32<float>(const float* v, uint32_t* w, float)
{
#pragma unroll
    for (int i = 0; i < 32; ++i) w[i] = __float_as_uint(v[i]);
}
template <> __device__ __forceinline__ void pack32<int8_t>(const float* v, uint32_t* w, float inv)
{
#pragma unroll
    for (int i = 0; i < 8; ++i) w[i] = nm_quant_i8x4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3], inv);
}

// v[0..31] += 32 residual values held as packed words
template <typename OutT> __device__ __forceinline__ void add_res32(const uint32_t* w, float* v);
template <> __device__ __forceinline__ void add_res32<__nv_bfloat16>(const uint32_t* w, float* v)
{
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[i]));
        v[2 * i] += f.x;
        v[2 * i + 1] += f.y;
    }
}
template <> __device__ __forceinline__ void add_res32<__half>(const uint32_t* w, float* v)
{
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
        v[2 * i] += f.x;
        v[2 * i + 1] += f.y;
    }
}
template <> __device__ __forceinline__ void add_res32<float>(const uint32_t* w, float* v)
{
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] += __uint_as_float(w[i]);
}
template <> __device__ __forceinline__ void add_res32<int8_t>(const uint32_t*, float*) {}

// First output pixel and image of patch p (convolution tiles).
struct Patch {
    int ox0, oy0, img0;
};
__device__ __forceinline__ Patch patch_of(const ConvDev& cv, int p)
{
    Patch r;
    const int tx = p % cv.tiles_x;
    const int rest = p / cv.tiles_x;
    r.ox0 = tx * cv.TW;
    r.oy0 = (rest % cv.tiles_y) * cv.TH;
    r.img0 = (rest / cv.tiles_y) * cv.NB;
    return r;
}

// Residual tile of one staging group: 32 rows x 128 bytes into `dst`, completion counted on `bar`.  The rows
// are matrix rows row0.. (linear operator) or the sub-box of patch `pt` that starts at patch row sub_h of its
// sub_n-th image (convolution); `col` is the group's first output column.
template <bool CONV>
__device__ __forceinline__ void res_tile_load(void* dst, const CUtensorMap* tmR, uint64_t* bar, int col, int row0,
                                              const Patch& pt, int sub_h, int sub_n)
{
    nm_mbar_expect_tx(bar, STAGE_BUF);
    if constexpr (CONV) nm_tma_load_4d(dst, tmR, col, pt.ox0, pt.oy0 + sub_h, pt.img0 + sub_n, bar);
    else nm_tma_load_2d(dst, tmR, col, row0, bar);
}

template <typename InT, typename OutT, bool TWO, int BN, bool CONV>
__global__ void __launch_bounds__(NUM_THREADS, 1)
linear_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                 const __grid_constant__ CUtensorMap tmO, const __grid_constant__ CUtensorMap tmR, const TcArgs a)
{
    static_assert(BN == 64 || BN == 128 || BN == 256, "tile widths built");
    constexpr int B_ROWS = TWO ? BN / 2 : BN;
    constexpr int B_BYTES = B_ROWS * ROW_BYTES;
    constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    constexpr int TILE_M = TWO ? 2 * BM : BM;
    constexpr int BK_ELEMS = ROW_BYTES / (int)sizeof(InT);
    constexpr uint32_t TMEM_COLS = 2 * BN;
    constexpr uint32_t IDESC = nm_idesc(TcIn<InT>::c_fmt, TcIn<InT>::ab_fmt, 0, 0, TILE_M, BN);
    // epilogue geometry: the two warps of a lane quarter split the tile's columns (BN/2 each), or, for the
    // 64-column tile, take alternate tiles (64 columns each).  A chunk is 32 columns; a staging group is 128
    // bytes of output per row: 64 columns of a 16-bit type, 32 of fp32, 128 of int8.
    constexpr bool ALT = BN == 64;
    constexpr int WCOLS = ALT ? 64 : BN / 2;                                 // columns a warp takes from a tile
    constexpr int NCH = WCOLS / 32;                                          // chunks per warp and tile
    constexpr int GC = sizeof(OutT) == 4 ? 1 : (sizeof(OutT) == 2 ? 2 : 4);  // chunks per group
    static_assert(NCH % GC == 0, "int8 output needs the 256-column tile");
    constexpr int NG = NCH / GC;                                             // groups per warp and tile
    constexpr int GROUP_COLS = 32 * GC;
    constexpr int WPC = 32 / GC;  // packed words per chunk
    constexpr int EPI_STEP = ALT ? 2 : 1;   // a warp works on every EPI_STEP-th tile of its CTA

    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_full[MAX_STAGES];
    __shared__ uint64_t bar_empty[MAX_STAGES];
    __shared__ uint64_t bar_acc_full[2];
    __shared__ uint64_t bar_acc_empty[2];
    __shared__ uint64_t bar_res[NUM_EPI_WARPS];
    __shared__ uint64_t bar_res_free[NUM_EPI_WARPS];
    __shared__ uint64_t bar_drain;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    const int stages = a.stages;
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* stage_out = tiles + (size_t)stages * STAGE_BYTES;   // 8 x 4 KB
    uint8_t* stage_res = stage_out + NUM_EPI_WARPS * STAGE_BUF;   // 8 x 4 KB when a residual is given
    float2* rep = reinterpret_cast<float2*>(stage_res + (a.has_res ? NUM_EPI_WARPS * STAGE_BUF : 0));
    // per epilogue warp: bias (128 floats) and, for int8, a_scale * w_scale (128 floats) of its tile columns
    float* vec_s = reinterpret_cast<float*>(rep + (size_t)a.n_seg * 32);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = TWO ? nm_cluster_ctarank() : 0u;  // 0 = leader of the pair
    const int tile_first = TWO ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int tile_step = TWO ? (int)(gridDim.x >> 1) : (int)gridDim.x;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        nm_prefetch_tmap(&tmA);
        nm_prefetch_tmap(&tmW);
        nm_prefetch_tmap(&tmO);
        if (a.has_res) nm_prefetch_tmap(&tmR);
        for (int s = 0; s < stages; ++s) {
            nm_mbar_init(&bar_full[s], 1);
            nm_mbar_init(&bar_empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            nm_mbar_init(&bar_acc_full[b], 1);
            nm_mbar_init(&bar_acc_empty[b], (ALT ? NUM_EPI_WARPS / 2 : NUM_EPI_WARPS) * (TWO ? 2 : 1));
        }
        for (int w = 0; w < NUM_EPI_WARPS; ++w) {
            nm_mbar_init(&bar_res[w], 1);
            nm_mbar_init(&bar_res_free[w], 32);
        }
        nm_mbar_init(&bar_drain, 1);
        nm_fence_barrier_init();
    }
    if (warp == 1) {
        if constexpr (TWO) {
            nm_tmem_alloc2(&tmem_slot, TMEM_COLS);
            nm_tmem_relinquish2();
        } else {
            nm_tmem_alloc(&tmem_slot, TMEM_COLS);
            nm_tmem_relinquish();
        }
    }
    if (a.tab) nm_table_replicate(rep, a.tab, a.n_seg, threadIdx.x, NUM_THREADS);
    nm_tc_fence_before();
    __syncthreads();
    if constexpr (TWO) nm_cluster_sync();  // both CTAs' barriers and tensor memory are ready
    nm_tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    volatile int* abortp = &abort_flag;
    // set-up done: the next kernel in the stream may begin its own set-up; nothing produced by the
    // previous kernel has been touched yet, everything below may depend on it
    nm_grid_launch_dependents();
    nm_grid_dependency_wait();

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        // All 32 lanes run the loop, so that stage, coordinates and addresses stay warp-uniform (the
        // compiler keeps them in uniform registers); one elected lane issues the copies.
        {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = tile_first; ok && tile < a.num_tiles; tile += tile_step) {
                const int mt = tile / a.num_n_tiles;
                const int m0 = mt * TILE_M + (int)rank * BM;
                const int n0 = (tile % a.num_n_tiles) * BN + (int)rank * B_ROWS;
                Patch pt = {0, 0, 0};
                if constexpr (CONV) pt = patch_of(a.cv, mt * (TWO ? 2 : 1) + (int)rank);
                int tap = 0, cb = 0;   // CONV: K-block = (tap, channel block)
                for (int kb = 0; kb < a.num_k_blocks; ++kb) {
                    if (!__all_sync(0xffffffffu, nm_mbar_wait(&bar_empty[stage], phase ^ 1u, abortp, a.status))) { ok = false; break; }
                    uint8_t* sa = tiles + (size_t)stage * STAGE_BYTES;
                    int c_c = 0, c_w = 0, c_h = 0, w_k = kb * BK_ELEMS, w_n = n0;
                    if constexpr (CONV) {
                        const int ky = tap / a.cv.kw_eff, kx = tap - ky * a.cv.kw_eff;
                        c_c = cb * BK_ELEMS;
                        c_w = pt.ox0 * a.cv.sw - a.cv.pw + kx;
                        c_h = pt.oy0 * a.cv.sh - a.cv.ph + ky;
                        if (a.cv.dw) {   // pooling: channel block = column tile, one constant matrix for every tap and tile
                            c_c = (tile % a.num_n_tiles) * BK_ELEMS;
                            w_k = 0;
                            w_n = (int)rank * B_ROWS;
                        }
                    }
                    if (nm_elect_one()) {
                        if constexpr (TWO) {
                            // both CTAs' copies are counted on the leader's barrier
                            const uint32_t full = nm_mapa(nm_smem_u32(&bar_full[stage]), 0);
                            if (rank == 0) nm_mbar_expect_tx(&bar_full[stage], 2 * STAGE_BYTES);
                            if constexpr (CONV) nm_tma_load_4d_2cta(sa, &tmA, c_c, c_w, c_h, pt.img0, full);
                            else nm_tma_load_2d_2cta(sa, &tmA, kb * BK_ELEMS, m0, full);
                            nm_tma_load_2d_2cta(sa + A_BYTES, &tmW, w_k, w_n, full);
                        } else {
                            nm_mbar_expect_tx(&bar_full[stage], STAGE_BYTES);
                            if constexpr (CONV) nm_tma_load_4d(sa, &tmA, c_c, c_w, c_h, pt.img0, &bar_full[stage]);
                            else nm_tma_load_2d(sa, &tmA, kb * BK_ELEMS, m0, &bar_full[stage]);
                            nm_tma_load_2d(sa + A_BYTES, &tmW, w_k, w_n, &bar_full[stage]);
                        }
                    }
                    __syncwarp();
                    if constexpr (CONV) {
                        if (++cb == a.cv.cblocks) { cb = 0; ++tap; }
                    }
                    if (++stage == stages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                long long t0 = clock64();  // bounded pause: copies in flight land before teardown
                while (clock64() - t0 < 4000000LL) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (the leader CTA of a pair)
        // All 32 lanes run the loop (waits, counters and descriptors stay warp-uniform); one elected
        // lane, always the same, issues the tcgen05 instructions and their commits.
        if (rank == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int buf = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            for (int tile = tile_first; ok && tile < a.num_tiles; tile += tile_step) {
                // CTA-scope acquire also where the peer CTA's epilogue warps arrive: what the hand-back orders are
                // tcgen05 operations, ordered by tcgen05.fence (a cluster-scope acquire costs ~400 cycles per tile)
                if (!__all_sync(0xffffffffu, nm_mbar_wait(&bar_acc_empty[buf], acc_phase ^ 1u, abortp, a.status))) { ok = false; break; }
                nm_tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                for (int kb = 0; kb < a.num_k_blocks; ++kb) {
                    if (!__all_sync(0xffffffffu, nm_mbar_wait(&bar_full[stage], phase, abortp, a.status))) { ok = false; break; }
                    nm_tc_fence_after();
                    const uint32_t sa = nm_smem_u32(tiles + (size_t)stage * STAGE_BYTES);
                    const uint64_t adesc = nm_smem_desc_sw128(sa);
                    const uint64_t bdesc = nm_smem_desc_sw128(sa + A_BYTES);
                    if (nm_elect_one()) {
#pragma unroll
                        for (int k = 0; k < 4; ++k) {  // 4 x 32 bytes of K per 128-byte row
                            const uint32_t accum = (kb | k) != 0 ? 1u : 0u;
                            if constexpr (TWO) {
                                if constexpr (TcIn<InT>::is_int) nm_mma_i8_2cta(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC, accum);
                                else nm_mma_f16_2cta(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC, accum);
                            } else {
                                if constexpr (TcIn<InT>::is_int) nm_mma_i8(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC, accum);
                                else nm_mma_f16(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC, accum);
                            }
                        }
                        // smem stage reusable (in both CTAs of a pair) once these MMAs retire
                        if constexpr (TWO) nm_tc_commit2(&bar_empty[stage], 3);
                        else nm_tc_commit(&bar_empty[stage]);
                    }
                    __syncwarp();
                    if (++stage == stages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (nm_elect_one()) {
                    if constexpr (TWO) nm_tc_commit2(&bar_acc_full[buf], 3);
                    else nm_tc_commit(&bar_acc_full[buf]);
                }
                __syncwarp();
                buf ^= 1;
                if (buf == 0) acc_phase ^= 1u;
            }
            if (!ok) {
                if (nm_elect_one()) {
                    if constexpr (TWO) nm_tc_commit2(&bar_drain, 1);
                    else nm_tc_commit(&bar_drain);
                    long long t0 = clock64();
                    while (!nm_mbar_try_wait(&bar_drain, 0) && clock64() - t0 < 200000000LL) {}
                }
                __syncwarp();
            }
        }
    } else {
        // ------------------------------------------------ epilogue (warps 2..9)
        const int e = warp - 2;   // epilogue warp index
        const int q = warp & 3;   // tensor-memory lane quarter this warp may read
        const int wsel = e >> 2;  // which of the quarter's two warps
        const int half = ALT ? 0 : wsel;            // which half of the tile's columns
        const int col_off = half * (BN / 2);        // first tile column of this warp
        uint8_t* my_out = stage_out + e * STAGE_BUF;
        uint8_t* my_res = stage_res + e * STAGE_BUF;
        const uint32_t my_out_row = nm_smem_u32(my_out) + (uint32_t)lane * 128u;
        const uint32_t my_res_row = nm_smem_u32(my_res) + (uint32_t)lane * 128u;
        const uint32_t rep_lane = nm_smem_u32(rep) + (uint32_t)lane * 8u;
        uint32_t res_phase = 0, res_free_phase = 0;
        const bool has_tab = a.tab != nullptr;
        const bool has_res = a.has_res != 0;
        const float inv_h = has_tab ? a.tab->inv_h : 0.f;
        const float off = has_tab ? a.tab->off : 0.f;
        const float nm1 = (float)(a.n_seg - 1);
        // the tiles this warp works on: every EPI_STEP-th of the CTA's, starting with its wsel-th
        const int my_first = tile_first + (ALT ? wsel * tile_step : 0);
        const int my_step = tile_step * EPI_STEP;
        // Where the 32 rows of this warp lie: rows q*32.. of the matrix tile, or (CONV) a sub-box of the patch.
        int sub_h = 0, sub_n = 0;   // CONV: first patch row / image of this warp's 32 tile rows
        if constexpr (CONV) {
            const int r0 = q * 32 / a.cv.TW;   // index of the warp's first (image, row) pair within the patch
            sub_h = r0 % a.cv.TH;
            sub_n = r0 / a.cv.TH;
        }
        const int row_base = (int)rank * BM + q * 32;   // first row of this warp within a tile's rows
        // residual of the first group of the first tile
        if (has_res && lane == 0 && my_first < a.num_tiles) {
            const int mt0 = my_first / a.num_n_tiles;
            Patch pt0 = {0, 0, 0};
            if constexpr (CONV) pt0 = patch_of(a.cv, mt0 * (TWO ? 2 : 1) + (int)rank);
            res_tile_load<CONV>(my_res, &tmR, &bar_res[e], (my_first % a.num_n_tiles) * BN + col_off, mt0 * TILE_M + row_base,
                                pt0, sub_h, sub_n);
        }
        int ok = 1;
        // All lanes test a barrier; only when it is not yet complete does lane 0 poll (with sleeps).
        auto wait_all = [&](uint64_t* bar, uint32_t par) {
            const bool done = nm_mbar_try_wait(bar, par);
            if (!__all_sync(0xffffffffu, done)) {
                int w = 1;
                if (lane == 0) w = nm_mbar_wait_relaxed(bar, par, abortp, a.status) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, w, 0);
                if (ok) (void)nm_mbar_try_wait(bar, par);  // every lane observes the phase itself
            }
        };
        // Per-column vectors of the warp's tile columns go through shared memory: lane l fetches
        // columns 4l..4l+3 one tile ahead (the latency hides behind the current tile), and the chunk
        // loop reads them as broadcasts.
        const bool use_vec = a.bias != nullptr || TcIn<InT>::is_int;
        float* my_vec = vec_s + e * 256;
        float4 nxt_b = make_float4(0.f, 0.f, 0.f, 0.f), nxt_s = make_float4(0.f, 0.f, 0.f, 0.f);
        auto fetch_vec = [&](int t) {
            nxt_b = make_float4(0.f, 0.f, 0.f, 0.f);
            nxt_s = make_float4(0.f, 0.f, 0.f, 0.f);
            if (!use_vec || t >= a.num_tiles || 4 * lane >= WCOLS) return;
            const int64_t col = (int64_t)(t % a.num_n_tiles) * BN + col_off + 4 * lane;
            if (col < a.N) {
                if (a.bias) nxt_b = __ldg(reinterpret_cast<const float4*>(a.bias + col));
                if constexpr (TcIn<InT>::is_int) {
                    const float4 ws = __ldg(reinterpret_cast<const float4*>(a.w_scale + col));
                    nxt_s = make_float4(a.a_scale * ws.x, a.a_scale * ws.y, a.a_scale * ws.z, a.a_scale * ws.w);
                }
            }
        };
        fetch_vec(my_first);
        // the CTA's it-th tile uses accumulator buffer it & 1, in that buffer's (it >> 1)-th use
        for (int tile = my_first, it = ALT ? wsel : 0; ok && tile < a.num_tiles; tile += my_step, it += EPI_STEP) {
            const int buf = it & 1;
            const uint32_t acc_phase = (uint32_t)((it >> 1) & 1);
            const int mt = tile / a.num_n_tiles;
            const int m0 = mt * TILE_M + (int)rank * BM;
            const int n0 = (tile % a.num_n_tiles) * BN + col_off;
            Patch pt = {0, 0, 0};
            if constexpr (CONV) pt = patch_of(a.cv, mt * (TWO ? 2 : 1) + (int)rank);
            if (use_vec) {
                __syncwarp();   // the previous tile's reads of my_vec are done
                *reinterpret_cast<float4*>(my_vec + 4 * lane) = nxt_b;
                if constexpr (TcIn<InT>::is_int) *reinterpret_cast<float4*>(my_vec + 128 + 4 * lane) = nxt_s;
                __syncwarp();
                fetch_vec(tile + my_step);
            }
            wait_all(&bar_acc_full[buf], acc_phase);
            if (!ok) break;
            nm_tc_fence_after();
            const int64_t row = (int64_t)m0 + q * 32 + lane;
            const bool row_ok = !CONV && row < a.M;
            bool store_rows;   // do this warp's 32 rows exist at all?
            if constexpr (CONV) store_rows = pt.oy0 + sub_h < a.cv.Ho && pt.img0 + sub_n < a.cv.Nimg;
            else store_rows = (int64_t)m0 + q * 32 < a.M;
            const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + col_off);
            uint32_t r[32];
#pragma unroll
            for (int g = 0; g < NG; ++g) {
                uint32_t packed[32];
                uint32_t rsv[32];
                if (has_res) {
                    wait_all(&bar_res[e], res_phase);
                    res_phase ^= 1u;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint32_t addr = my_res_row + (uint32_t)((c ^ (lane & 7)) << 4);
                        asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];"
                                     : "=r"(rsv[4 * c]), "=r"(rsv[4 * c + 1]), "=r"(rsv[4 * c + 2]), "=r"(rsv[4 * c + 3])
                                     : "r"(addr)
                                     : "memory");
                    }
                    // The buffer is refilled by the TMA unit, which is not ordered with this warp's shared-memory
                    // reads by program order or by a warp barrier: every lane releases the buffer on a barrier
                    // of its own (the arrival is ordered after the lane's reads), lane 0 acquires all 32
                    // arrivals and only then issues the copy.
                    nm_mbar_arrive(&bar_res_free[e]);
                    if (lane == 0) ok = nm_mbar_wait(&bar_res_free[e], res_free_phase, abortp, a.status) ? ok : 0;
                    res_free_phase ^= 1u;
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    // the buffer is free again: fetch the residual of the next group (this tile's, or
                    // the first group of this warp's next tile) while this one is computed
                    if (lane == 0 && ok) {
                        int nmt = mt, ncol = n0 + (g + 1) * GROUP_COLS;
                        bool more = true;
                        if (g + 1 == NG) {
                            const int nt = tile + my_step;
                            more = nt < a.num_tiles;
                            nmt = nt / a.num_n_tiles;
                            ncol = (nt % a.num_n_tiles) * BN + col_off;
                        }
                        if (more) {
                            Patch npt = pt;
                            if constexpr (CONV) {
                                if (nmt != mt) npt = patch_of(a.cv, nmt * (TWO ? 2 : 1) + (int)rank);
                            }
                            res_tile_load<CONV>(my_res, &tmR, &bar_res[e], ncol, nmt * TILE_M + row_base, npt, sub_h, sub_n);
                        }
                    }
                }
#pragma unroll
                for (int cc = 0; cc < GC; ++cc) {
                    const int c = g * GC + cc;
                    // Load and wait in one statement.  Keeping the next chunk's load in flight across this chunk's
                    // arithmetic measured no faster (the quarter's other warp covers the latency), and registers
                    // with a load in flight are not safe from compiler-made copies until the wait.
                    nm_tmem_ld32_sync(t_addr + (uint32_t)(c * 32), r);
                    if (c + 1 == NCH) {
                        // this warp's share of the accumulator is in registers: hand the buffer back
                        nm_tc_fence_before();
                        __syncwarp();
                        if (lane == 0) {
                            if constexpr (TWO) nm_mbar_arrive_cluster(nm_mapa(nm_smem_u32(&bar_acc_empty[buf]), 0));
                            else nm_mbar_arrive(&bar_acc_empty[buf]);
                        }
                        __syncwarp();
                    }
                    const int64_t col0 = (int64_t)n0 + c * 32;
                    float v[32];
                    // columns beyond N are computed on zero operands and clipped by the TMA store;
                    // only the loads of bias / scale and the debug dumps need the bound
                    if constexpr (TcIn<InT>::is_int) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4) {
                            // a_scale * w_scale and bias of columns beyond N are zero
                            const float4 ws = *reinterpret_cast<const float4*>(my_vec + 128 + c * 32 + i);
                            const float4 bs = *reinterpret_cast<const float4*>(my_vec + c * 32 + i);
                            if (a.acc_dump && row_ok && col0 + i < a.N)
                                *reinterpret_cast<int4*>(a.acc_dump + row * a.N + col0 + i) =
                                    make_int4((int)r[i], (int)r[i + 1], (int)r[i + 2], (int)r[i + 3]);
                            uint64_t d01, d23;   // fma((float)acc, scale, bias), two columns per packed instruction
                            asm("fma.rn.f32x2 %0, %1, %2, %3;"
                                : "=l"(d01)
                                : "l"(nm_pack2((float)(int)r[i], (float)(int)r[i + 1])), "l"(nm_pack2(ws.x, ws.y)), "l"(nm_pack2(bs.x, bs.y)));
                            asm("fma.rn.f32x2 %0, %1, %2, %3;"
                                : "=l"(d23)
                                : "l"(nm_pack2((float)(int)r[i + 2], (float)(int)r[i + 3])), "l"(nm_pack2(ws.z, ws.w)),
                                  "l"(nm_pack2(bs.z, bs.w)));
                            nm_unpack2(d01, v[i], v[i + 1]);
                            nm_unpack2(d23, v[i + 2], v[i + 3]);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
                        if (a.bias) {
#pragma unroll
                            for (int i = 0; i < 32; i += 4) {   // zero beyond N; two columns per packed add
                                const float4 bs = *reinterpret_cast<const float4*>(my_vec + c * 32 + i);
                                uint64_t s01, s23;
                                asm("add.rn.f32x2 %0, %1, %2;" : "=l"(s01) : "l"(nm_pack2(v[i], v[i + 1])), "l"(nm_pack2(bs.x, bs.y)));
                                asm("add.rn.f32x2 %0, %1, %2;" : "=l"(s23) : "l"(nm_pack2(v[i + 2], v[i + 3])), "l"(nm_pack2(bs.z, bs.w)));
                                nm_unpack2(s01, v[i], v[i + 1]);
                                nm_unpack2(s23, v[i + 2], v[i + 3]);
                            }
                        }
                    }
                    if (has_res && a.res_first) add_res32<OutT>(&rsv[cc * WPC], v);
                    if (has_tab) {
                        if (a.idx_dump) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) {
                                int s;
                                v[i] = nm_pwl_fast(rep_lane, v[i], inv_h, off, nm1, &s);
                                if (row_ok && col0 + i < a.N) a.idx_dump[row * a.N + col0 + i] = s;
                            }
                        } else {
                            const uint64_t inv_h2 = nm_pack2(inv_h, inv_h), off2 = nm_pack2(off, off);
#pragma unroll
                            for (int i = 0; i < 32; i += 2) nm_pwl_fast2(rep_lane, v[i], v[i + 1], inv_h2, off2, nm1);
                        }
                    } else if (a.idx_dump) {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (row_ok && col0 + i < a.N) a.idx_dump[row * a.N + col0 + i] = -1;
                    }
                    if (has_res && !a.res_first) add_res32<OutT>(&rsv[cc * WPC], v);
                    pack32<OutT>(v, &packed[cc * WPC], a.inv_out_scale);
                }
                // stage the group and send it: the previous store must have finished reading the buffer
                if (lane == 0) nm_tma_store_wait_read();
                __syncwarp();
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint32_t addr = my_out_row + (uint32_t)((c ^ (lane & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(packed[4 * c]),
                                 "r"(packed[4 * c + 1]), "r"(packed[4 * c + 2]), "r"(packed[4 * c + 3])
                                 : "memory");
                }
                nm_fence_proxy_async();
                __syncwarp();
                // a group that lies wholly beyond the matrix is not stored at all
                if (lane == 0 && ok && n0 + g * GROUP_COLS < a.N && store_rows) {
                    if constexpr (CONV) nm_tma_store_4d(&tmO, my_out, n0 + g * GROUP_COLS, pt.ox0, pt.oy0 + sub_h, pt.img0 + sub_n);
                    else nm_tma_store_2d(&tmO, my_out, n0 + g * GROUP_COLS, m0 + q * 32);
                }
            }
        }
        if (lane == 0) nm_tma_store_wait_read();  // staging memory must outlive the last store's reads
        __syncwarp();
    }

    // ---------------------------------------------------- teardown (all paths)
    nm_tc_fence_before();
    __syncthreads();
    if constexpr (TWO) nm_cluster_sync();  // the peer may still use barriers / tensor memory of the pair
    if (warp == 1) {
        __syncwarp();
        nm_tc_fence_after();
        if constexpr (TWO) nm_tmem_dealloc2(tmem_base, TMEM_COLS);
        else nm_tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline CUtensorMapDataType tmap_type(nm_dtype dt)
{
    return dt == NM_BF16  ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
           : dt == NM_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
           : dt == NM_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                          : CU_TENSOR_MAP_DATA_TYPE_UINT8;
}

// 2-D row-major matrix [rows, cols] with row pitch ld (elements); box = 128 bytes x box_rows, 128-byte swizzle.
inline nm_status make_tmap(nm_ctx* ctx, CUtensorMap* m, const void* base, nm_dtype dt, int64_t rows, int64_t cols,
                           int64_t ld, int box_rows)
{
    const size_t es = nm_dtype_size(dt);
    cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t gstr[1] = {(cuuint64_t)ld * es};
    cuuint32_t box[2] = {(cuuint32_t)(ROW_BYTES / es), (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = ((EncodeTiledFn)ctx->encode_tiled)(m, tmap_type(dt), 2, const_cast<void*>(base), gdim, gstr, box, estr,
                                                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? NM_OK : NM_ERR_CUDA;
}

// Shared-memory bytes and stage count of one launch; false if the kernel cannot run with this table size.
template <typename InT, bool TWO, int BN>
inline bool plan_smem(TcArgs* a, bool has_vec, size_t* smem_out)
{
    constexpr int B_ROWS = TWO ? BN / 2 : BN;
    constexpr int STAGE_BYTES = A_BYTES + B_ROWS * ROW_BYTES;
    const size_t table_bytes = (size_t)a->n_seg * 32 * sizeof(float2);
    const size_t vec_bytes = has_vec ? (size_t)NUM_EPI_WARPS * 256 * sizeof(float) : 0;
    const size_t staging = (size_t)NUM_EPI_WARPS * STAGE_BUF * (a->has_res ? 2 : 1) + vec_bytes;
    const size_t budget = 227 * 1024 - 1024 /*alignment slack*/ - 1024 /*static*/ - table_bytes - staging;
    int stages = (int)(budget / STAGE_BYTES);
    if (stages > MAX_STAGES) stages = MAX_STAGES;
    if (stages < 2) return false;
    a->stages = stages;
    *smem_out = (size_t)stages * STAGE_BYTES + staging + table_bytes + 1024;
    return true;
}

// Launches the persistent kernel over a.num_tiles tiles (one CTA, or one CTA pair, per resident slot).
template <typename InT, typename OutT, bool TWO, int BN, bool CONV>
inline nm_status launch_kernel(nm_ctx* ctx, const CUtensorMap& tmA, const CUtensorMap& tmW, const CUtensorMap& tmO,
                               const CUtensorMap& tmR, const TcArgs& a, size_t smem, double work, cudaStream_t st)
{
    auto kern = linear_tc_kernel<InT, OutT, TWO, BN, CONV>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return NM_ERR_CUDA;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    cfg.attrs = attr;
    cfg.numAttrs = 0;
    if (ctx->pdl) {
        attr[cfg.numAttrs].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[cfg.numAttrs].val.programmaticStreamSerializationAllowed = 1;
        cfg.numAttrs++;
    }
    if constexpr (TWO) {
        attr[cfg.numAttrs].id = cudaLaunchAttributeClusterDimension;
        attr[cfg.numAttrs].val.clusterDim.x = 2;
        attr[cfg.numAttrs].val.clusterDim.y = 1;
        attr[cfg.numAttrs].val.clusterDim.z = 1;
        cfg.numAttrs++;
        // persistent: no more clusters than can be resident at once (cached per kernel and smem size)
        static int max_clusters = 0;
        static size_t max_clusters_smem = 0;
        if (max_clusters == 0 || max_clusters_smem != smem) {
            cfg.gridDim = dim3(2 * (unsigned)(ctx->sm_count / 2));
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n < 1) return NM_ERR_CUDA;
            max_clusters = n;
            max_clusters_smem = smem;
        }
        const int pairs = a.num_tiles < max_clusters ? a.num_tiles : max_clusters;
        cfg.gridDim = dim3(2 * (unsigned)pairs);
    } else {
        cfg.gridDim = dim3((unsigned)(a.num_tiles < ctx->sm_count ? a.num_tiles : ctx->sm_count));
    }
    NmLaunchScope scope(ctx, NM_KERNEL_LINEAR_TC, work, st);
    if (cudaLaunchKernelEx(&cfg, kern, tmA, tmW, tmO, tmR, a) != cudaSuccess) return NM_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? NM_OK : NM_ERR_CUDA;
}

}  // namespace nm_tc
